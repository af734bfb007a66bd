// Fast rotate+quantize kernel: rows of d = G * 1024 channels.
//   b <= 128              every scale mode (INT4 per token / per 128, MXFP4, FP4 per token, asymmetric
//                         INT4 per token), with or without a permutation (permuted: d <= 16384);
//   b in {256, 512, 1024} unpermuted, INT4 per token or MXFP4;
//   b == d <= 8192        unpermuted, INT4 per token or MXFP4 (full-vector rotation).
// Per-token scales need G <= 15 (one named barrier per group of G warps).
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
// (normally one) look for the exact value.  Normally one slot holds it: its position is
// recorded and the scale is stored later, 32 records at a time, one per lane (see "deferred
// per-token scales" below).  Otherwise the exact values are derived at once; with one such
// warp it stores the scale itself, with several the last one to add its value to a shared
// accumulator does.  Warps that need the exact maximum for a tie fix-up (rare) wait for its
// publication (a value, or the position to evaluate) on a flag, with a bounded spin.
//
// Asymmetric INT4 per token: the warps exchange signed maxima and minima.  Normally one warp holds the
// candidates for the row maximum and one (maybe the same) those for the minimum, each in one slot: the
// two positions are published and recorded, and the step and the zero point (exact extremes from global
// memory, three fp64 divisions) are derived 32 rows at a time, one per lane.  A side with several slots
// publishes its exact value instead of a position; a row with several candidate warps on a side combines
// exact values through two shared accumulators.  A warp that needs (s, z) for a fix-up evaluates the
// published pair itself.  The zero point is subtracted inside the magic constant of the rounding trick,
// so the low nibble of the sum is the unsigned code; where rounding min / step in fp32 is a close call
// the row waits for the exact pair before it quantises.
//
// Permuted rows are staged raw and gathered by every warp into its own 2 KB buffer; blocks
// longer than 128 continue the butterfly across lane groups (shuffles) and, for b == d,
// across the warps of the row (shared-memory exchange).
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
constexpr float FAST_ERR_K = 4.0f;          // fp32 error model: |u32 - u| <= K * log2(b) * 2^-24 * max|u32| of the block
constexpr float FAST_ERR_K_LONG = 2.0f;     // blocks of 256 and 512
constexpr float FAST_ERR_K_FULL = 1.0f;     // whole-row blocks: 4096 outputs share the rounding errors of 12 stages
constexpr uint32_t WAIT_SPIN_LIMIT = 1u << 22;

// per-token INT4, INT4 per 128, MXFP4, and E2M1 with a per-token fp32 scale (the scale logic of MODE_TOKEN
// with the element conversion of MODE_MX)
// MODE_ASYM: asymmetric INT4 per token (step and integer zero point from the row's signed extremes)
enum FastMode { MODE_TOKEN = 0, MODE_G128 = 1, MODE_MX = 2, MODE_FP4 = 3, MODE_ASYM = 4 };
__host__ __device__ constexpr bool per_token_mode(int mode) { return mode == MODE_TOKEN || mode == MODE_FP4 || mode == MODE_ASYM; }

struct FastParams {
    const uint16_t *x;
    uint8_t *out_codes;
    void *out_scales;
    uint32_t units_total;    // units of G segments (fewer than 2^31); rows when G = d / 1024
    const uint16_t *x2;      // gated-activation variants only: the second projection ("up"), same shape as x
    const int32_t *perm;     // permuted variants only: perm[d] (device)
    int G;                   // permuted variants: segments per row
    int d;
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
    static constexpr size_t wacc2 = wpub + (size_t)FAST_WARPS * 2 * 8;              // asymmetric: the same two for the row minimum
    static constexpr size_t wpub2 = wacc2 + (size_t)FAST_WARPS * 2 * 8;             //   (and the published zero point)
    static constexpr size_t wmax = wpub2 + (size_t)FAST_WARPS * 2 * 8;              // [2][FAST_WARPS] f32 warp maxima
    static constexpr size_t wmin = wmax + (size_t)FAST_WARPS * 2 * 4;               // [2][FAST_WARPS] f32 warp minima (asymmetric)
    static constexpr size_t wcnt = wmin + (size_t)FAST_WARPS * 2 * 4;               // [2][FAST_WARPS] u32 arrival counts
    static constexpr size_t wflag = wcnt + (size_t)FAST_WARPS * 2 * 4;              // [2][FAST_WARPS] u32 publication flags
    static constexpr size_t wreq = wflag + (size_t)FAST_WARPS * 2 * 4;              // [FAST_WARPS][32] u64 deferred scale requests
    static constexpr size_t wreq2 = wreq + (size_t)FAST_WARPS * 32 * 8;             // asymmetric: [FAST_WARPS][32] u64 second key of a record
    static constexpr size_t wrequ = wreq2 + (size_t)FAST_WARPS * 32 * 8;            //   and [FAST_WARPS][32] u32 its row
    static constexpr size_t empty = wrequ + (size_t)FAST_WARPS * 32 * 4;            // [FAST_WARPS * FAST_NSTAGE] mbarriers
    static constexpr size_t used = empty + (size_t)FAST_WARPS * FAST_NSTAGE * 8;
    static constexpr size_t total = used + 1024;                                    // room to align the base
    // permuted variants: the stage area holds 3 raw-row stages per group (96 KB in all) followed by
    // one permuted 2 KB segment per warp; the permutation (as 16-bit byte offsets) follows `used`
    static constexpr size_t pbuf = stages + (size_t)FAST_WARPS * 3 * SEG_BYTES;
    static constexpr size_t perm_tab = used;
    static constexpr int PERM_MAX_D = 16384;
    static constexpr size_t total_perm = used + (size_t)PERM_MAX_D * 2 + 1024;
    // full-vector variants (unpermuted): 3 stages as well, and 4 KB per warp of fp32 exchange space after `used`
    static constexpr size_t xbuf = used;
    static constexpr size_t total_full = used + (size_t)FAST_WARPS * 4096 + 1024;
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
// The common case costs one poll; the bounded loop is entered only when that poll fails.
__device__ __forceinline__ bool mbar_wait_fast(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0u || mbar_wait(bar, parity);
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Programmatic dependent launch: a kernel launched with programmatic stream serialization may start while
// its predecessor in the stream is still running; it must not touch global memory before griddep_wait(),
// which returns once the predecessor has completed and its writes are visible (at once when there is none,
// or when the launch did not ask for the overlap).  griddep_launch() lets the successor's CTAs be scheduled
// as soon as this grid's CTAs have all passed it or exited.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
template <int OFF>
__device__ __forceinline__ void ldmatrix_x4_at(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4+%5];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr), "n"(OFF));
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
template <int OFF>
__device__ __forceinline__ void sts_u16_at(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u16 [%0+%2], %1;" ::"r"(addr), "h"((uint16_t)v), "n"(OFF) : "memory");
}
// Store of the 16-bit code piece of slot s (a constant once the slot loop is unrolled) at base ^ (s * 8),
// for a base whose offset bits 3..5 lie inside XV: the slot bits in XV are XORed into the address, the
// others are added as an immediate offset (no instruction).
template <int XV>
__device__ __forceinline__ void sts_code(uint32_t base, int s, uint32_t v)
{
    const uint32_t a = base ^ (uint32_t)((s & XV) * 8);
    switch (s & ~XV & 7) {
    case 0: sts_u16_at<0>(a, v); break;
    case 1: sts_u16_at<8>(a, v); break;
    case 2: sts_u16_at<16>(a, v); break;
    case 3: sts_u16_at<24>(a, v); break;
    case 4: sts_u16_at<32>(a, v); break;
    case 5: sts_u16_at<40>(a, v); break;
    case 6: sts_u16_at<48>(a, v); break;
    default: sts_u16_at<56>(a, v); break;
    }
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts_v4f(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void lds_v4f(uint32_t addr, float &a, float &b, float &c, float &d)
{
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(a), "=f"(b), "=f"(c), "=f"(d) : "r"(addr) : "memory");
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
__device__ __forceinline__ float warp_min_f32(float v)
{
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
// double <-> 64-bit key with the same order (keys of finite values are never 0 or all ones)
__device__ __forceinline__ unsigned long long order_key(double f)
{
    const unsigned long long u = (unsigned long long)__double_as_longlong(f);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
__device__ __forceinline__ double order_value(unsigned long long k)
{
    return __longlong_as_double((long long)((k >> 63) ? (k & 0x7fffffffffffffffull) : ~k));
}
// max over the warp of a non-negative double, on its bit pattern (or of any 64-bit key)
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v)
{
    const uint32_t hi = __reduce_max_sync(0xffffffffu, (uint32_t)(v >> 32));
    const uint32_t lo = __reduce_max_sync(0xffffffffu, ((uint32_t)(v >> 32) == hi) ? (uint32_t)v : 0u);
    return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ float max3abs(float acc, float a, float b) { return fmaxf(fmaxf(acc, fabsf(a)), fabsf(b)); }

// Four fp32 values -> 16 bits of four E2M1 codes (first operand in the lowest nibble), RNE, saturating.
__device__ __forceinline__ uint32_t cvt_e2m1x4(float a, float b, float c, float d)
{
    uint32_t r;
    asm("{ .reg .b8 t0, t1; .reg .b32 w0, w1; cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1; cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3; "
        "cvt.u32.u8 w0, t0; cvt.u32.u8 w1, t1; mad.lo.u32 %0, w1, 256, w0; }" : "=r"(r) : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}

// Eight fp32 values -> two sets of four E2M1 codes in one word: bits 0..15 from (a0..a3), bits 16..31 from
// (b0..b3), first operand of a set in its lowest nibble.
__device__ __forceinline__ uint32_t cvt_e2m1x4_pair(float a0, float a1, float a2, float a3, float b0, float b1, float b2, float b3)
{
    uint32_t r;
    asm("{ .reg .b8 t0, t1, t2, t3; cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1; cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3; "
        "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5; cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7; mov.b32 %0, {t0, t1, t2, t3}; }"
        : "=r"(r) : "f"(a0), "f"(a1), "f"(a2), "f"(a3), "f"(b0), "f"(b1), "f"(b2), "f"(b3));
    return r;
}

__device__ __forceinline__ uint32_t hadamard_bf16(int k, int n) { return (__popc(k & n) & 1) ? 0xBF80u : 0x3F80u; }

// ---------------------------------------------------------------- exact re-evaluation

// bf16 bit pattern (low 16 bits of h) -> double, exactly, with integer operations (the
// fp32->fp64 conversion instruction is slow); zero and subnormals take the conversion.
__device__ __forceinline__ double bf16_bits_to_f64(uint32_t h)
{
    const uint32_t mag = h & 0x7fffu;
    if (mag < 0x80u) return (double)__uint_as_float(h << 16);
    return __hiloint2double((int)(((mag << 13) + 0x38000000u) | ((h & 0x8000u) << 16)), 0);
}

// Exact unnormalised output i of the block starting at `blk` (bf16 in shared memory), evaluated
// by the 4 lanes of a quad: each lane reduces a quarter of the block with a signed pairwise
// tree in fp64, then the quarters are combined.  q = lane % 4, qmask = the quad's lanes.
template <int LOG2B>
__device__ __forceinline__ double exact_coord_quad(const uint16_t *blk, int i, int q, unsigned qmask)
{
    constexpr int PER = (1 << LOG2B) / 4;
    double v[PER];
    const uint32_t *src = reinterpret_cast<const uint32_t *>(blk + q * PER);
#pragma unroll
    for (int r = 0; r < PER / 2; ++r) {
        const uint32_t w = src[r];
        v[2 * r] = bf16_bits_to_f64(w);
        v[2 * r + 1] = bf16_bits_to_f64(w >> 16);
    }
#pragma unroll
    for (int t = 0; (1 << t) < PER; ++t) {
        const double sg = ((i >> t) & 1) ? -1.0 : 1.0;
#pragma unroll
        for (int m = 0; m < (PER >> (t + 1)); ++m) v[m] = fma(sg, v[2 * m + 1], v[2 * m]);
    }
    double part = (__popc(i & (q << (LOG2B - 2))) & 1) ? -v[0] : v[0];
    part += __shfl_xor_sync(qmask, part, 1);
    part += __shfl_xor_sync(qmask, part, 2);
    return part;
}

// Exact unnormalised output i of the B-element block at blk, by a whole warp.
template <int B>
__device__ __forceinline__ double exact_coord_fast(const uint16_t *blk, int i, int lane)
{
    double acc = 0.0;
#pragma unroll(B <= 128 ? 4 : 8)
    for (int k0 = 0; k0 < B; k0 += 32) {
        const int k = k0 + lane;
        if (B >= 32 || k < B) {
            const double v = bf16_bits_to_f64(blk[k]);
            acc += (__popc(i & k) & 1) ? -v : v;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

// Exact unnormalised outputs i0 .. i0+3 (i0 a multiple of 4) of the B-element block at blk, by a
// whole warp: lane l returns output i0 + (l & 3).  Every lane adds its terms signed by the high
// bits of the output index; lanes with equal l & 3 are summed, then a 4-point butterfly over
// l & 3 applies the low two index bits.
template <int B>
__device__ __forceinline__ double exact_coord4(const uint16_t *blk, int i0, int lane)
{
    double acc = 0.0;
#pragma unroll(B <= 128 ? 4 : 8)
    for (int k0 = 0; k0 < B; k0 += 32) {
        const int k = k0 + lane;
        if (B >= 32 || k < B) {
            const double v = bf16_bits_to_f64(blk[k]);
            acc += (__popc(i0 & k) & 1) ? -v : v;
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    acc += __shfl_xor_sync(0xffffffffu, acc, 8);
    acc += __shfl_xor_sync(0xffffffffu, acc, 16);
#pragma unroll
    for (int bit = 1; bit <= 2; bit <<= 1) {
        const double other = __shfl_xor_sync(0xffffffffu, acc, bit);
        acc = (lane & bit) ? other - acc : acc + other;
    }
    return acc;
}

// The same for a permuted row: term k of the block is raw[off[k] / 2], with off the 16-bit byte
// offsets of the permutation, already advanced to the block's first position.
template <int B>
__device__ __forceinline__ double exact_coord4_perm(const uint16_t *raw, const uint16_t *off, int i0, int lane)
{
    double acc = 0.0;
#pragma unroll
    for (int k0 = 0; k0 < B; k0 += 32) {
        const int k = k0 + lane;
        if (B >= 32 || k < B) {
            const double v = bf16_bits_to_f64(raw[off[k] >> 1]);
            acc += (__popc(i0 & k) & 1) ? -v : v;
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    acc += __shfl_xor_sync(0xffffffffu, acc, 8);
    acc += __shfl_xor_sync(0xffffffffu, acc, 16);
#pragma unroll
    for (int bit = 1; bit <= 2; bit <<= 1) {
        const double other = __shfl_xor_sync(0xffffffffu, acc, bit);
        acc = (lane & bit) ? other - acc : acc + other;
    }
    return acc;
}

// Long blocks: the whole warp evaluates one record.  Lane l takes the 8 consecutive inputs
// 256 r + 8 l .. + 7 of every 256 (coalesced 16-byte loads), keeps the four partial sums by k & 3,
// and the lanes are summed before the 4-point butterfly.  Returns the largest magnitude of the
// four outputs i0 .. i0 + 3 (the same in every lane).
template <int B, bool GLOBAL>
__device__ __forceinline__ double exact_slot_max_wide(const uint16_t *blk, uint32_t i0, int lane)
{
    static_assert(B >= 256, "one 16-byte load per lane covers 256 inputs");
    double S[4] = {0.0, 0.0, 0.0, 0.0};
    const uint4 *src = reinterpret_cast<const uint4 *>(blk) + lane;
#pragma unroll(B / 256 < 16 ? B / 256 : 16)
    for (int r = 0; r < B / 256; ++r) {
        const uint4 w4 = GLOBAL ? __ldg(src + r * 32) : src[r * 32];
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
        const uint32_t k0 = (uint32_t)(r * 256 + lane * 8);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t flip = (__popc(i0 & (k0 + 4u * h)) & 1) ? 0x80008000u : 0u;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t word = w[2 * h + (e >> 1)] ^ flip;
                S[e] += bf16_bits_to_f64((e & 1) ? (word >> 16) : word);
            }
        }
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) S[m] += __shfl_xor_sync(0xffffffffu, S[m], o);
    }
    const double a0 = S[0] + S[1], a1 = S[0] - S[1], a2 = S[2] + S[3], a3 = S[2] - S[3];
    return fmax(fmax(fabs(a0 + a2), fabs(a1 + a3)), fmax(fabs(a0 - a2), fabs(a1 - a3)));
}

// Element e = s*4 + j of lane (g, q): block start (in elements, segment relative) and index inside the block.
template <int LOG2B>
__device__ __forceinline__ void locate(int g, int q, int e, int &blk_elem, int &i, int &elem)
{
    constexpr int CB = LOG2B - 4;                 // chunk bits inside a block
    constexpr int PM = (1 << CB) - 1;
    const int s = e >> 2, j = e & 3;
    const int p = g * 8 + (s ^ ((g & 3) & ~PM));  // chunk position inside the segment
    elem = p * 16 + 4 * q + j;
    blk_elem = (p >> CB) << LOG2B;
    i = elem - blk_elem;
}

// Bit mask of the lane's 32 held values (bit s*4+j) whose magnitude reaches thr; ms[s] is the
// magnitude maximum of slot s, used to skip slots.
__device__ __forceinline__ uint32_t candidate_mask(const f32x2 (&v)[8][2], const float (&ms)[8], float thr)
{
    uint32_t cm = 0u;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        if (ms[s] >= thr) {
            const float a = v[s][0].x, b = v[s][0].y, c = v[s][1].x, d = v[s][1].y;
            cm |= (fabsf(a) >= thr ? 1u : 0u) << (4 * s);
            cm |= (fabsf(b) >= thr ? 2u : 0u) << (4 * s);
            cm |= (fabsf(c) >= thr ? 4u : 0u) << (4 * s);
            cm |= (fabsf(d) >= thr ? 8u : 0u) << (4 * s);
        }
    }
    return cm;
}

// Exact maximum magnitude (bit pattern of a non-negative double, the same in every lane) over the
// slots of this warp's segment whose fp32 maximum reaches thr.
// FULL_LOG2 == 0: blocks of 2^LOG2B inside the segment at seg.  FULL_LOG2 > 0: blocks of 2^FULL_LOG2
// elements of the unit (row or segment) at seg, of which this warp's segment starts at seg_off.
template <int LOG2B, int FULL_LOG2>
__device__ __forceinline__ unsigned long long exact_max_of_candidates(const uint16_t *seg, int seg_off, const float (&ms)[8],
                                                                      float thr, int lane)
{
    constexpr int CB = LOG2B - 4;
    constexpr int PM = (1 << CB) - 1;
    uint32_t slot_mask = 0u;
#pragma unroll
    for (int s = 0; s < 8; ++s) slot_mask |= (ms[s] >= thr) ? (1u << s) : 0u;
    double best = 0.0;
    unsigned cw = __ballot_sync(0xffffffffu, slot_mask != 0u);
    while (cw) {
        const int src = __ffs(cw) - 1;
        cw &= cw - 1;
        uint32_t sm = __shfl_sync(0xffffffffu, slot_mask, src);
        const int sg = src >> 2;
        while (sm) {
            const int sl = __ffs(sm) - 1;
            sm &= sm - 1;
            const int pch = sg * 8 + (sl ^ ((sg & 3) & ~PM));      // chunk position in the segment
            if (FULL_LOG2 > 0) {
                const int pr = seg_off + pch * 16 + 4 * (src & 3), be = (pr >> FULL_LOG2) << FULL_LOG2;
                if (FULL_LOG2 >= 8)
                    best = fmax(best, exact_slot_max_wide<(1 << (FULL_LOG2 >= 8 ? FULL_LOG2 : 8)), false>(seg + be, (uint32_t)(pr - be), lane));
                else
                    best = fmax(best, fabs(exact_coord4<(1 << (FULL_LOG2 > 0 ? FULL_LOG2 : 4))>(seg + be, pr - be, lane)));
            } else {
                const int blk_elem = (pch >> CB) << LOG2B;
                const int i0 = pch * 16 - blk_elem + 4 * (src & 3);
                best = fmax(best, fabs(exact_coord4<(1 << LOG2B)>(seg + blk_elem, i0, lane)));
            }
        }
    }
    return warp_max_u64((unsigned long long)__double_as_longlong(best));
}

// ---------------------------------------------------------------- deferred per-token scales
//
// A per-token scale needs the exact magnitude of the row's largest rotated value.  In the common
// case the fp32 pass pins that value down to one slot (four adjacent outputs of one 16-element
// chunk).  The warp that owns the slot only records (row, position); when 32 records have
// gathered, each lane of the warp serves one of them on its own: it re-reads the block's b bf16
// inputs from global memory (64 to 256 bytes, usually still in L2), forms the four outputs in
// fp64 and stores the scale.  This costs a few instructions per row instead of a cooperative
// evaluation on the row's critical path.
//
// Record: bits 63..32 = index of a 1024-element segment, bits 15..0 = element offset from that
// segment's start to the slot's first output (per token: first segment of the row, offset in the row).
// The same scheme serves the per-128 scales, with one record per quad.

constexpr int WIDE_LOG2B = 10;      // blocks from this length on are served by the whole warp

template <int LOG2B, bool PERM>
__device__ __forceinline__ double exact_slot_max_global(const uint16_t *row, uint32_t pos, const int32_t *perm, int d)
{
    constexpr int B = 1 << LOG2B;
    const uint32_t blk = (pos >> LOG2B) << LOG2B;
    const uint32_t i0 = pos - blk;                       // multiple of 4
    const uint4 *src = reinterpret_cast<const uint4 *>(row + blk);
    double S[4] = {0.0, 0.0, 0.0, 0.0};                  // sums of the terms with k & 3 == m, signed by the high bits of i0
#pragma unroll(B <= 128 ? B / 8 : 2)
    for (int c = 0; c < B / 8; ++c) {
        uint32_t w[4];
        if (PERM) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int s0 = min(max(__ldg(perm + blk + 8 * c + 2 * e), 0), d - 1);
                const int s1 = min(max(__ldg(perm + blk + 8 * c + 2 * e + 1), 0), d - 1);
                w[e] = (uint32_t)__ldg(row + s0) | ((uint32_t)__ldg(row + s1) << 16);
            }
        } else {
            const uint4 w4 = __ldg(src + c);
            w[0] = w4.x; w[1] = w4.y; w[2] = w4.z; w[3] = w4.w;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const bool neg = __popc(i0 & (uint32_t)(8 * c + 4 * h)) & 1;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t word = w[2 * h + (e >> 1)];
                const double val = (double)__uint_as_float((e & 1) ? (word & 0xffff0000u) : (word << 16));
                S[e] += neg ? -val : val;
            }
        }
    }
    const double a0 = S[0] + S[1], a1 = S[0] - S[1], a2 = S[2] + S[3], a3 = S[2] - S[3];
    return fmax(fmax(fabs(a0 + a2), fabs(a1 + a3)), fmax(fabs(a0 - a2), fabs(a1 - a3)));
}

template <int LOG2B, int MODE, bool PERM>
__device__ __forceinline__ void serve_scale_requests(const FastParams &p, const unsigned long long *req, uint32_t n, int lane)
{
    __syncwarp();
    if (LOG2B >= WIDE_LOG2B && !PERM) {
        // long blocks: the whole warp evaluates one record at a time (coalesced reads)
        for (uint32_t j = 0; j < n; ++j) {
            const unsigned long long r = req[j];
            const uint32_t segi = (uint32_t)(r >> 32), off = (uint32_t)r & 0xffffu;
            const uint32_t segs = (uint32_t)p.d / SEG_ELEMS;
            const uint32_t row = segi / segs;
            const uint32_t pos = (segi - row * segs) * SEG_ELEMS + off;
            const uint32_t blk = (pos >> LOG2B) << LOG2B;
            const double a = exact_slot_max_wide<(1 << (LOG2B >= 8 ? LOG2B : 8)), true>(p.x + (size_t)row * p.d + blk, pos - blk, lane);
            if (lane == 0) {
                const size_t si = per_token_mode(MODE) ? (size_t)row : ((size_t)row * p.d + pos) >> 7;
                reinterpret_cast<float *>(p.out_scales)[si] = (a == 0.0) ? 0.0f : (float)(a * p.inv_7_sqrt_b);
            }
        }
        __syncwarp();
        return;
    }
    if ((uint32_t)lane < n) {
        const unsigned long long r = req[lane];
        const uint32_t segi = (uint32_t)(r >> 32), off = (uint32_t)r & 0xffffu;
        const uint32_t segs = (uint32_t)p.d / SEG_ELEMS;
        const uint32_t row = segi / segs;
        const uint32_t pos = (segi - row * segs) * SEG_ELEMS + off;      // position in the row
        const double a = exact_slot_max_global<LOG2B, PERM>(p.x + (size_t)row * p.d, pos, p.perm, p.d);
        const size_t si = per_token_mode(MODE) ? (size_t)row : ((size_t)row * p.d + pos) >> 7;
        reinterpret_cast<float *>(p.out_scales)[si] = (a == 0.0) ? 0.0f : (float)(a * p.inv_7_sqrt_b);
    }
    __syncwarp();
}

// Asymmetric INT4: step and zero point from the order keys of the exact unnormalised extremes, in the
// operation order of the definition (y = u / sqrt(b); s = (max y - min y) / 15; z = rne(min y / s)).
__device__ __forceinline__ void asym_step_zero(unsigned long long khi, unsigned long long klo, double sqrt_b, double &s64, double &z64)
{
    const double mxy = order_value(khi) / sqrt_b, mny = order_value(klo) / sqrt_b;
    s64 = (mxy - mny) / 15.0;
    z64 = (s64 == 0.0) ? 0.0 : rint(mny / s64);
}

// Signed maximum and minimum of the four outputs of one slot (position pos in the row, a multiple of 4),
// re-derived by one thread from the row in global memory (the signed counterpart of exact_slot_max_global).
template <int LOG2B, bool PERM>
__device__ __forceinline__ void exact_slot_extremes_global(const uint16_t *row, uint32_t pos, const int32_t *perm, int d,
                                                           double &mx, double &mn)
{
    constexpr int B = 1 << LOG2B;
    const uint32_t blk = (pos >> LOG2B) << LOG2B;
    const uint32_t i0 = pos - blk;
    const uint4 *src = reinterpret_cast<const uint4 *>(row + blk);
    double S[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll(B <= 128 ? B / 8 : 2)
    for (int c = 0; c < B / 8; ++c) {
        uint32_t w[4];
        if (PERM) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int s0 = min(max(__ldg(perm + blk + 8 * c + 2 * e), 0), d - 1);
                const int s1 = min(max(__ldg(perm + blk + 8 * c + 2 * e + 1), 0), d - 1);
                w[e] = (uint32_t)__ldg(row + s0) | ((uint32_t)__ldg(row + s1) << 16);
            }
        } else {
            const uint4 w4 = __ldg(src + c);
            w[0] = w4.x; w[1] = w4.y; w[2] = w4.z; w[3] = w4.w;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const bool neg = __popc(i0 & (uint32_t)(8 * c + 4 * h)) & 1;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t word = w[2 * h + (e >> 1)];
                const double val = (double)__uint_as_float((e & 1) ? (word & 0xffff0000u) : (word << 16));
                S[e] += neg ? -val : val;
            }
        }
    }
    const double a0 = S[0] + S[1], a1 = S[0] - S[1], a2 = S[2] + S[3], a3 = S[2] - S[3];
    const double o0 = a0 + a2, o1 = a1 + a3, o2 = a0 - a2, o3 = a1 - a3;
    mx = fmax(fmax(o0, o1), fmax(o2, o3));
    mn = fmin(fmin(o0, o1), fmin(o2, o3));
}

// An entry of an asymmetric record is the order key of an exact extreme (always >= 2^52) or, below 2^32,
// the position in the row of the one slot that holds it.
__device__ __forceinline__ bool asym_entry_is_position(unsigned long long e) { return e < (1ull << 32); }

// Deferred (s, z) of up to 32 rows, one per lane: positions are evaluated from global memory, and the three
// divisions cost a few hundred instructions, which a lane per row amortises over the warp.
template <int LOG2B, bool PERM>
__device__ __forceinline__ void serve_asym_requests(const FastParams &p, const unsigned long long *ehi, const unsigned long long *elo,
                                                    const uint32_t *rows, uint32_t n, int lane)
{
    __syncwarp();
    if ((uint32_t)lane < n) {
        unsigned long long khi = ehi[lane], klo = elo[lane];
        const uint16_t *row = p.x + (size_t)rows[lane] * p.d;
        if (asym_entry_is_position(khi)) {
            double mx, mn;
            exact_slot_extremes_global<LOG2B, PERM>(row, (uint32_t)khi, p.perm, p.d, mx, mn);
            if (asym_entry_is_position(klo) && klo == khi) klo = order_key(mn);
            khi = order_key(mx);
        }
        if (asym_entry_is_position(klo)) {
            double mx, mn;
            exact_slot_extremes_global<LOG2B, PERM>(row, (uint32_t)klo, p.perm, p.d, mx, mn);
            klo = order_key(mn);
        }
        double s64, z64;
        asym_step_zero(khi, klo, p.sqrt_b, s64, z64);
        float2 *dst = reinterpret_cast<float2 *>(p.out_scales) + rows[lane];
        *dst = make_float2((float)s64, (float)z64);
    }
    __syncwarp();
}

// ---------------------------------------------------------------- gated activation in front of the rotation
//
// h = Swish(g) * u, Swish(g) = g / (1 + exp(-g)), rounded once to bf16 (round to nearest even): the input of the
// online rotation in a gated feedforward block.  The fp32 evaluation below works on pairs (packed fp32
// instructions) and is accurate to 11 * 2^-24 = 6.6e-7 relative wherever no intermediate leaves the normal
// range: exp2 of a compensated argument (2^-22 for the approximation, 2^-24 each for the correction factor and
// its product; weighted by e / (1 + e) <= 1), the sum 1 + e (2^-24), one approximate reciprocal (2^-23), two
// products (2^-24 each).  A result whose low half-word lies in
// [0x7fe0, 0x801f] -- within 31 fp32 ulps, at least 1.8e-6 relative, of the halfway pattern 0x8000 -- could
// round to either neighbour and is evaluated again in fp64; so is every result that is zero, below 2^-100 or
// not finite, which covers the arguments whose exponential or reciprocal left the normal range (they give a
// zero or an infinity here) and the subnormal results, where the relative bound does not hold.
__device__ __forceinline__ float ex2_ftz(float x)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float rcp_ftz(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ f32x2 swish_mul2(f32x2 g, f32x2 u)
{
    const float L2E_HI = 1.44269502162933349609375f, L2E_LO = 1.925963033500011e-8f;      // log2(e) = hi + lo
    const float LN2 = 0.693147182464599609375f;
    const f32x2 tp = mul2(g, pack2(L2E_HI, L2E_HI));                 // -t, rounded
    f32x2 r = fma2(g, pack2(-L2E_HI, -L2E_HI), tp);                  // t_exact - t: what the rounding dropped
    r = fma2(g, pack2(-L2E_LO, -L2E_LO), r);
    f32x2 e = pack2(ex2_ftz(-tp.x), ex2_ftz(-tp.y));
    // 2^(t + r) = 2^t (1 + r ln 2) to first order (|r| < 2^-17); as a product, so that an infinite 2^t stays one
    e = mul2(e, fma2(r, pack2(LN2, LN2), pack2(1.0f, 1.0f)));
    const f32x2 den = add2(e, pack2(1.0f, 1.0f));
    const f32x2 rc = pack2(rcp_ftz(den.x), rcp_ftz(den.y));
    return mul2(mul2(g, rc), u);                                     // (finite inputs never give a NaN in this order)
}
// zero if and only if the low half-word of an fp32 pattern lies in [0x7fe0, 0x801f]
__device__ __forceinline__ uint32_t swiglu_midpoint_key(float h) { return ((__float_as_uint(h) + 0x20u) & 0xffc0u) ^ 0x8000u; }
__device__ __forceinline__ bool swiglu_needs_fp64(float h)
{
    return swiglu_midpoint_key(h) == 0u || !(fabsf(h) >= 0x1p-100f) || !(fabsf(h) <= 3.4028234663852886e38f);
}
// A finite double to bf16 bits, one rounding to nearest even (integer arithmetic on the double's fields).
__device__ __forceinline__ uint32_t double_to_bf16_bits(double v)
{
    const unsigned long long b = (unsigned long long)__double_as_longlong(v);
    const uint32_t sign = (uint32_t)(b >> 48) & 0x8000u;
    const int E = (int)((b >> 52) & 0x7ffu);
    if (E == 0) return sign;                                   // zero (fp64 subnormals are far below bf16's)
    const int e = E - 1023;
    if (e > 127) return sign | 0x7f80u;
    const unsigned long long M = (1ull << 52) | (b & ((1ull << 52) - 1ull));
    const int lead = e < -126 ? -126 : e;
    const int shift = 45 + (lead - e);                         // the quantum is 2^(lead - 7)
    if (shift > 54) return sign;                               // below half of the smallest subnormal
    unsigned long long q = M >> shift;
    const unsigned long long rem = M & ((1ull << shift) - 1ull), half = 1ull << (shift - 1);
    if (rem > half || (rem == half && (q & 1ull))) q += 1ull;
    const uint32_t mag = (e >= -126) ? (uint32_t)((e + 127) << 7) + (uint32_t)(q - 128ull) : (uint32_t)q;
    return sign | (mag > 0x7f80u ? 0x7f80u : mag);
}
__device__ __noinline__ uint32_t swiglu_fp64_bits(float g, float u)
{
    if (g == 0.0f || u == 0.0f) return ((__float_as_uint(g) ^ __float_as_uint(u)) >> 16) & 0x8000u;      // a signed zero
    const double gd = (double)g;
    return double_to_bf16_bits(gd / (1.0 + exp(-gd)) * (double)u);
}
// Eight values of h (one 16-byte piece, four words of two bf16) from the matching pieces of the projections.
// The three reasons for the fp64 route are reduced over the piece (one integer minimum, the smallest and the
// largest magnitude) and tested once.
__device__ __forceinline__ void swiglu_piece(const uint32_t (&gw)[4], const uint32_t (&uw)[4], uint32_t (&hw)[4])
{
    f32x2 h[4];
    uint32_t key = 0xffffffffu;
    float lo = 3.0e38f, hi = 0.0f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const f32x2 g = pack2(__uint_as_float(gw[k] << 16), __uint_as_float(gw[k] & 0xffff0000u));
        const f32x2 u = pack2(__uint_as_float(uw[k] << 16), __uint_as_float(uw[k] & 0xffff0000u));
        h[k] = swish_mul2(g, u);
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hw[k]) : "f"(h[k].y), "f"(h[k].x));
        key = min(key, min(swiglu_midpoint_key(h[k].x), swiglu_midpoint_key(h[k].y)));
        lo = fminf(fminf(lo, fabsf(h[k].x)), fabsf(h[k].y));
        hi = fmaxf(fmaxf(hi, fabsf(h[k].x)), fabsf(h[k].y));
    }
    if (key == 0u || !(lo >= 0x1p-100f) || !(hi <= 3.4028234663852886e38f)) {       // rare
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (swiglu_needs_fp64(h[k].x))
                hw[k] = (hw[k] & 0xffff0000u) | swiglu_fp64_bits(__uint_as_float(gw[k] << 16), __uint_as_float(uw[k] << 16));
            if (swiglu_needs_fp64(h[k].y))
                hw[k] = (hw[k] & 0x0000ffffu) |
                        (swiglu_fp64_bits(__uint_as_float(gw[k] & 0xffff0000u), __uint_as_float(uw[k] & 0xffff0000u)) << 16);
        }
    }
}
// This warp's 1024-element segment of h, written over the staged gate segment (lane l handles the 16-byte
// pieces l, l + 32, l + 64, l + 96 of both projections).
__device__ __forceinline__ void swiglu_segment(uint32_t gate_addr, uint32_t up_addr, int lane)
{
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t off = (uint32_t)(r * 32 + lane) * 16u;
        uint32_t gw[4], uw[4];
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(gw[0]), "=r"(gw[1]), "=r"(gw[2]), "=r"(gw[3]) : "r"(gate_addr + off) : "memory");
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(uw[0]), "=r"(uw[1]), "=r"(uw[2]), "=r"(uw[3]) : "r"(up_addr + off) : "memory");
        uint32_t hw[4];
        swiglu_piece(gw, uw, hw);
        sts_v4(gate_addr + off, hw[0], hw[1], hw[2], hw[3]);
    }
    __syncwarp();
}

// ---------------------------------------------------------------- the kernel

// XB > 0: the Hadamard block has 2^(7 + XB) elements (LOG2B must be 7: the part of the
// butterfly done inside a warp's registers); the lane-group bits go through shuffles, the warp bits
// through shared memory.
// XB = 1..3 keeps the block inside a warp's segment; XB = 3 + LOG2G is the whole row.
// SWIGLU: the rows are h = Swish(x) * x2, formed in shared memory from the two staged projections (unpermuted,
// blocks inside a segment); two ring stages of each projection instead of four of one, and no deferred scales
// (they would be re-derived from the inputs in global memory, which are not h).
template <int LOG2B, int MODE, int LOG2G, bool PERM, int XB, bool SWIGLU = false>
__global__ void __launch_bounds__(FAST_THREADS, 1) perq_fast_kernel(FastParams p)
{
    static_assert(!SWIGLU || (!PERM && XB == 0 && MODE != MODE_ASYM && MODE != MODE_FP4), "gated variant: unpermuted, short blocks");
    constexpr int B = 1 << LOG2B;
    constexpr bool FULLV = XB > 0;                           // a block longer than the in-register part
    constexpr int WBITS = XB > 3 ? XB - 3 : 0;               // index bits that span the warps of a row
    constexpr int LBITS = XB > 3 ? 3 : XB;                   // index bits that span the lane groups of a warp
    constexpr int LOG2BF = FULLV ? 7 + XB : LOG2B;           // log2 of the Hadamard block
    static_assert(WBITS == 0 || WBITS == LOG2G, "blocks that span warps are whole rows");
    constexpr int BF = 1 << LOG2BF;
    static_assert(!FULLV || (LOG2B == 7 && !PERM && MODE != MODE_G128), "full-vector variant: unpermuted, per token or MX");
    constexpr int CB = LOG2B - 4;                 // butterfly stages left after the tensor-core H_16
    constexpr int PM = (1 << CB) - 1;             // slot bits inside a Hadamard block
    constexpr int NCLS = (PM & 3) + 1;            // sign classes of the slot relabelling
    // G is a template constant 2^LOG2G, or (LOG2G < 0, and permuted rows without per-token scales) p.G
    constexpr bool TOK = per_token_mode(MODE);
    constexpr bool RUNTIME_G = (PERM && !TOK) || LOG2G < 0;
    constexpr int NST = (PERM || WBITS > 0) ? 3 : SWIGLU ? 2 : FAST_NSTAGE;
    const int G = RUNTIME_G ? p.G : (1 << (LOG2G < 0 ? 0 : LOG2G));   // warps (segments) per unit
    const int GROUPS = FAST_WARPS / G;
    const uint32_t UNIT_BYTES = (uint32_t)G * SEG_BYTES;
    constexpr float MAGIC = 12582920.0f;          // 1.5 * 2^23 + 8: low nibble of the sum = code + 8
    static_assert(TOK || LOG2G == 0 || WBITS > 0, "only per-token scales or a full-vector block couple the warps of a row");
    extern __shared__ __align__(128) unsigned char fsmem_raw[];
    // 1024-byte aligned base: the ldmatrix and code-store addresses below are formed with XOR
    unsigned char *fsmem = fsmem_raw + ((1024u - (smem_u32(fsmem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int group = RUNTIME_G ? warp / G : warp >> (LOG2G < 0 ? 0 : LOG2G);
    // Position of this warp in its row group, rotated by the group index.  Warps are handed to the SM's four
    // schedulers by warp index, and for many inputs the same position of every row does the extra per-row
    // work (the segment that holds the outlier channel finds the exact maximum; position 0 issues the
    // loads): without the rotation those warps of all groups would share one scheduler.
    const int w_in_g = (warp - group * G + group) % G;
    const unsigned qmask = 0xFu << (lane & 28);
    const float err_rel = (!FULLV ? FAST_ERR_K : LOG2BF >= 10 ? FAST_ERR_K_FULL : FAST_ERR_K_LONG) * (float)LOG2BF * TWO_M24;
    // u / sqrt(b) as the definition computes it.  For an even log2(b) the divisor is a power of two: the
    // product with its reciprocal is the same double and spares the fix-ups an fp64 division.
    auto over_sqrt_b = [&](double u) -> double {
        return (LOG2BF % 2 == 0) ? u * (1.0 / (double)(1 << (LOG2BF / 2))) : u / p.sqrt_b;
    };
    const uint32_t xbuf_addr = smem_u32(fsmem + FastSmem::xbuf) + (uint32_t)(group * G) * 4096u;   // FULLV: this row's exchange space

    const uint32_t stage_base = smem_u32(fsmem + FastSmem::stages) + (uint32_t)group * (NST * UNIT_BYTES);
    // gated variant: the second projection's stages fill the other half of the stage area
    const uint32_t up_base = stage_base + (uint32_t)FAST_WARPS * 2u * SEG_BYTES;
    const uint32_t empty_base = smem_u32(fsmem + FastSmem::empty) + (uint32_t)group * (FAST_NSTAGE * 8);
    const uint32_t pbuf_addr = smem_u32(fsmem + FastSmem::pbuf) + (uint32_t)warp * SEG_BYTES;
    const uint16_t *ptab = reinterpret_cast<const uint16_t *>(fsmem + FastSmem::perm_tab);
    const uint32_t code_base = smem_u32(fsmem + FastSmem::codes) + (uint32_t)warp * (2 * SEG_CODE_BYTES);
    const uint32_t full_base = smem_u32(fsmem + FastSmem::full) + (uint32_t)group * (FAST_NSTAGE * 8);
    unsigned long long *wacc = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wacc);
    unsigned long long *wpub = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wpub);
    float *wmax = reinterpret_cast<float *>(fsmem + FastSmem::wmax);
    float *wmin = reinterpret_cast<float *>(fsmem + FastSmem::wmin);
    unsigned long long *wacc2 = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wacc2);
    unsigned long long *wpub2 = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wpub2);
    uint32_t *wcnt = reinterpret_cast<uint32_t *>(fsmem + FastSmem::wcnt);
    uint32_t *wflag = reinterpret_cast<uint32_t *>(fsmem + FastSmem::wflag);
    unsigned long long *wreq = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wreq) + warp * 32;
    unsigned long long *wreq2 = reinterpret_cast<unsigned long long *>(fsmem + FastSmem::wreq2) + warp * 32;
    uint32_t *wrequ = reinterpret_cast<uint32_t *>(fsmem + FastSmem::wrequ) + warp * 32;
    uint32_t nreq = 0;                       // records waiting in wreq (the same in every lane)
    const bool leader = (w_in_g == 0) && (lane == 0);

    if (tid < FAST_WARPS * FAST_NSTAGE) {
        mbar_init(smem_u32(fsmem + FastSmem::full) + tid * 8, 1);
        if (PERM) mbar_init(smem_u32(fsmem + FastSmem::empty) + tid * 8, (uint32_t)G);
    }
    griddep_wait();             // nothing above reads or writes global memory
    griddep_launch();           // the stream's next kernel may be set up on every SM this grid has left (it waits like this one)
    if (PERM) {     // the permutation as byte offsets into a staged row; out-of-range entries are clamped
        uint16_t *pt = reinterpret_cast<uint16_t *>(fsmem + FastSmem::perm_tab);
        if ((reinterpret_cast<uintptr_t>(p.perm) & 15u) == 0) {      // four entries per load, all loads independent
            const int4 *p4 = reinterpret_cast<const int4 *>(p.perm);
#pragma unroll 8
            for (int i = tid; i < p.d / 4; i += FAST_THREADS) {
                const int4 e = __ldg(p4 + i);
                const uint32_t o0 = (uint32_t)(2 * min(max(e.x, 0), p.d - 1)), o1 = (uint32_t)(2 * min(max(e.y, 0), p.d - 1));
                const uint32_t o2 = (uint32_t)(2 * min(max(e.z, 0), p.d - 1)), o3 = (uint32_t)(2 * min(max(e.w, 0), p.d - 1));
                reinterpret_cast<uint2 *>(pt)[i] = make_uint2(o0 | (o1 << 16), o2 | (o3 << 16));
            }
        } else {
            for (int i = tid; i < p.d; i += FAST_THREADS) pt[i] = (uint16_t)(2 * min(max(__ldg(p.perm + i), 0), p.d - 1));
        }
    }
    if (tid < 2 * FAST_WARPS) { wacc[tid] = 0ull; wacc2[tid] = ~0ull; wcnt[tid] = 0u; wflag[tid] = 0u; }
    if (tid == 0) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    const uint32_t first = blockIdx.x * GROUPS + group;
    const uint32_t stride = gridDim.x * GROUPS;
    if (group >= GROUPS || first >= p.units_total) return;   // whole groups leave together (no barrier is shared across groups)

    // Hadamard operand of the tensor-core stage: column n of MMA m is output 4*(n/2) + (n%2) + 2m.
    uint32_t hb[2][2];
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        const int col = 4 * (g >> 1) + (g & 1) + 2 * m;
        hb[m][0] = hadamard_bf16(2 * q, col) | (hadamard_bf16(2 * q + 1, col) << 16);
        hb[m][1] = hadamard_bf16(2 * q + 8, col) | (hadamard_bf16(2 * q + 9, col) << 16);
    }
    // ldmatrix source offset of tile 0: lane l feeds row (l & 7) of matrix (l >> 3); slot 2t + (mi & 1)
    // of lane group r8 comes from chunk r8*8 + (slot ^ f), halves swapped when r8 & 4.  Tile t is at
    // this offset XOR (t << 6).
    uint32_t lm0;
    {
        const int r8 = lane & 7, mi = lane >> 3;
        const int f = r8 & 3, fh = (r8 >> 2) & 1;
        lm0 = (uint32_t)((r8 * 8 + ((mi & 1) ^ f)) * 32 + (((mi >> 1) ^ fh) * 16));
    }
    const int f_g = g & 3;
    // byte offset of this lane's 16-bit code piece of slot 0 inside the segment's 512 code bytes;
    // slot s is at this offset XOR (s * 8)
    const uint32_t code_lane = (uint32_t)((g * 8 + (f_g & ~PM)) * 8 + 2 * q);
    // sign of the held value relative to the true output, per (s & 3 & PM): folded into multipliers
    const float half_sign = ((g & 4) && q >= 2) ? -1.0f : 1.0f;
    float sgn[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) sgn[k] = (__popc(k & f_g & PM) & 1) ? -half_sign : half_sign;
    // sign to fold into the quantisation multiplier of class k (none once the true signs are restored)
    auto qsgn = [&](int k) { return FULLV ? 1.0f : sgn[k]; };

    // This group's units are first, first + stride, ...: n_units of them.  Addresses advance by increments
    // (the loop is bound by the number of instructions it issues).
    const uint32_t n_units = (p.units_total - first + stride - 1) / stride;
    const uint32_t refill_end = n_units > (uint32_t)NST ? n_units - NST : 0u;      // iterations 1 .. refill_end load a unit
    const size_t unit_step = (size_t)stride * ((size_t)G * SEG_ELEMS);
    const uint16_t *xload = p.x + (size_t)first * ((size_t)G * SEG_ELEMS);         // leader: the next unit to load
    const uint16_t *xload2 = (SWIGLU ? p.x2 : p.x) + (size_t)first * ((size_t)G * SEG_ELEMS);
    // prologue: fill the ring
    if (leader) {
#pragma unroll
        for (int s = 0; s < NST; ++s) {
            if ((uint32_t)s < n_units) {
                mbar_expect_tx(full_base + s * 8, SWIGLU ? 2 * UNIT_BYTES : UNIT_BYTES);
                bulk_load(stage_base + s * UNIT_BYTES, xload, UNIT_BYTES, full_base + s * 8);
                if (SWIGLU) bulk_load(up_base + s * UNIT_BYTES, xload2, UNIT_BYTES, full_base + s * 8);
                xload += unit_step;
                xload2 += unit_step;
            }
        }
    }
    // quantisation multipliers of the sign classes, up to the scale range's factor (a sign change is exact, so
    // inv * (sgn * (1 +- delta)) are the same floats as (sgn * inv) * (1 +- delta))
    const float q_delta = 16.0f * err_rel + 5.0e-7f;
    float q_cp[NCLS], q_cm[NCLS];
#pragma unroll
    for (int k = 0; k < NCLS; ++k) { q_cp[k] = qsgn(k) * (1.0f + q_delta); q_cm[k] = qsgn(k) * (1.0f - q_delta); }

    uint8_t *code_out = p.out_codes + ((size_t)first * G + w_in_g) * SEG_CODE_BYTES;   // this warp's codes of the current unit
    const size_t code_out_step = (size_t)stride * G * SEG_CODE_BYTES;
    uint32_t unit = first;
    for (uint32_t it = 0; it < n_units; ++it, unit += stride, code_out += code_out_step) {
        const uint32_t stage = it % NST;
        const uint32_t parity = (it / NST) & 1u;
        const uint32_t par2 = it & 1u;
        if (!mbar_wait_fast(full_base + stage * 8, parity)) {
            // the load never completed: every warp of the group polls this barrier and leaves here together,
            // so none is left behind at the group's named barrier
            if (lane == 0) atomicOr(&g_perq_device_error, 1u);
            bulk_store_wait_read<0>();
            return;
        }
        // the staged row (or, unpermuted, the staged unit) and this warp's 1024 elements of it
        const uint16_t *raw_row = reinterpret_cast<const uint16_t *>(fsmem + FastSmem::stages) +
                                  ((size_t)group * NST + stage) * ((size_t)G * SEG_ELEMS);
        uint32_t seg_addr = stage_base + stage * UNIT_BYTES + (uint32_t)w_in_g * SEG_BYTES;
        const uint16_t *seg = raw_row + (size_t)w_in_g * SEG_ELEMS;
        if (SWIGLU) swiglu_segment(seg_addr, up_base + stage * UNIT_BYTES + (uint32_t)w_in_g * SEG_BYTES, lane);
        if (PERM) {
            // gather this warp's segment of the permuted row into its own buffer: lane l takes
            // positions r*256 + 8l .. +7 in round r (16-byte conflict-free stores)
            const uint32_t raw_addr = stage_base + stage * UNIT_BYTES;
            const uint4 *offs = reinterpret_cast<const uint4 *>(ptab + (size_t)w_in_g * SEG_ELEMS) + lane;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint4 o = offs[r * 32];
                const uint32_t ow[4] = {o.x, o.y, o.z, o.w};
                uint32_t wv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    wv[e] = lds_u16(raw_addr + (ow[e] & 0xffffu)) | (lds_u16(raw_addr + (ow[e] >> 16)) << 16);
                sts_v4(pbuf_addr + (uint32_t)(r * 512 + lane * 16), wv[0], wv[1], wv[2], wv[3]);
            }
            __syncwarp();
            seg_addr = pbuf_addr;
            seg = reinterpret_cast<const uint16_t *>(fsmem + FastSmem::pbuf) + (size_t)warp * SEG_ELEMS;
        }
        const size_t seg_index = (size_t)unit * G + w_in_g;
        // Hadamard block of the element at offset e of this warp's segment: its bf16 inputs and the
        // element's index inside the block
        auto block_of = [&](int e, const uint16_t *&bp, int &i) {
            if (FULLV) {
                const int er = w_in_g * SEG_ELEMS + e, be = (er >> LOG2BF) << LOG2BF;
                bp = raw_row + be;
                i = er - be;
            } else {
                const int be = (e >> LOG2B) << LOG2B;
                bp = seg + be;
                i = e - be;
            }
        };

        // ---- H_16 on the tensor cores; v[s][h] = outputs (2h, 2h+1) of this lane's four of slot s
        f32x2 v[8][2];
        auto h16_tensor = [&](f32x2 (&w)[8][2]) {
            const uint32_t a0 = seg_addr + lm0;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                uint32_t a[4];
                // (bit 7 of the lane's offset is clear: tile bit 1 is an immediate offset, tile bit 0 an XOR)
                if (t & 2) ldmatrix_x4_at<128>(a, a0 ^ (uint32_t)((t & 1) << 6));
                else ldmatrix_x4_at<0>(a, a0 ^ (uint32_t)((t & 1) << 6));
                float c0[4], c1[4];
                mma_bf16(c0, a, hb[0][0], hb[0][1]);
                mma_bf16(c1, a, hb[1][0], hb[1][1]);
                w[2 * t][0] = pack2(c0[0], c0[1]);
                w[2 * t][1] = pack2(c1[0], c1[1]);
                w[2 * t + 1][0] = pack2(c0[2], c0[3]);
                w[2 * t + 1][1] = pack2(c1[2], c1[3]);
            }
        };
        // the butterfly stages over the slot bits inside a block (packed add/sub)
        auto slot_stages = [&](f32x2 (&w)[8][2]) {
#pragma unroll
            for (int t = 0; t < CB; ++t) {
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    if ((s & (1 << t)) == 0) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const f32x2 a = w[s][h], c = w[s | (1 << t)][h];
                            w[s][h] = add2(a, c);
                            w[s | (1 << t)][h] = sub2(a, c);
                        }
                    }
                }
            }
        };
        h16_tensor(v);
        // refill the stage the previous iteration used (every warp of the group is past it now:
        // for G == 1 because this warp is, for G > 1 after the named barrier below)
        auto refill = [&]() {
            if (leader && it - 1u < refill_end) {        // it >= 1 and unit it + NST - 1 exists (it - 1 wraps for it == 0)
                const uint32_t ps = (it - 1) % NST;
                // permuted rows are read until the end of an iteration: wait until every warp is done
                if (PERM && !mbar_wait(empty_base + ps * 8, ((it - 1) / NST) & 1u)) atomicOr(&g_perq_device_error, 4u);
                mbar_expect_tx(full_base + ps * 8, SWIGLU ? 2 * UNIT_BYTES : UNIT_BYTES);
                bulk_load(stage_base + ps * UNIT_BYTES, xload, UNIT_BYTES, full_base + ps * 8);
                if (SWIGLU) bulk_load(up_base + ps * UNIT_BYTES, xload2, UNIT_BYTES, full_base + ps * 8);
                xload += unit_step;
                xload2 += unit_step;
            }
        };
        if (G == 1 || (!TOK && WBITS == 0)) refill();

        // ---- remaining butterfly stages over the slot bits inside a block
        slot_stages(v);

        if (FULLV) {
            // ---- the rest of a full-vector butterfly.  First the true signs (the relabelling signs
            // can no longer be folded into a multiplier once values of different lanes are mixed).
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const f32x2 sg2 = pack2(sgn[s & 3], sgn[s & 3]);
                v[s][0] = mul2(v[s][0], sg2);
                v[s][1] = mul2(v[s][1], sg2);
            }
            // lane-group bits (chunk index bits 3..5): exchange with lanes 4, 8, 16 away
#pragma unroll
            for (int bit = 4; bit < (4 << LBITS); bit <<= 1) {
                const float sg = (lane & bit) ? -1.0f : 1.0f;
                const f32x2 sg2 = pack2(sg, sg);
#pragma unroll
                for (int s = 0; s < 8; ++s) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const f32x2 o = pack2(__shfl_xor_sync(0xffffffffu, v[s][h].x, bit),
                                              __shfl_xor_sync(0xffffffffu, v[s][h].y, bit));
                        v[s][h] = fma2(v[s][h], sg2, o);          // upper partner: other - mine, lower: mine + other
                    }
                }
            }
            // warp bits (segment index): through shared memory, every warp combines all G copies
            if (WBITS > 0) {
                const uint32_t mine = xbuf_addr + (uint32_t)w_in_g * 4096u + (uint32_t)lane * 16u;
#pragma unroll
                for (int s = 0; s < 8; ++s) sts_v4f(mine + s * 512, v[s][0].x, v[s][0].y, v[s][1].x, v[s][1].y);
                named_barrier(1 + group, G * 32);
                refill();
                {
                    const float sg = (__popc(w_in_g) & 1) ? -1.0f : 1.0f;
                    const f32x2 sg2 = pack2(sg, sg);
#pragma unroll
                    for (int s = 0; s < 8; ++s) { v[s][0] = mul2(v[s][0], sg2); v[s][1] = mul2(v[s][1], sg2); }
                }
#pragma unroll
                for (int dw = 1; dw < (1 << WBITS); ++dw) {
                    const int wo = w_in_g ^ dw;                   // every other warp of the row once
                    const float sg = (__popc(w_in_g & wo) & 1) ? -1.0f : 1.0f;
                    const f32x2 sg2 = pack2(sg, sg);
                    const uint32_t theirs = xbuf_addr + (uint32_t)wo * 4096u + (uint32_t)lane * 16u;
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        float a, b, c, d;
                        lds_v4f(theirs + s * 512, a, b, c, d);
                        v[s][0] = fma2(pack2(a, b), sg2, v[s][0]);
                        v[s][1] = fma2(pack2(c, d), sg2, v[s][1]);
                    }
                }
            }
        }

        // ---- fp32 maxima per slot
        // (per token and MX only need them in rare paths and recompute them there: fewer live registers)
        float ms[8];
        auto slot_maxima = [&]() {
#pragma unroll
            for (int s = 0; s < 8; ++s) ms[s] = fmaxf(max3abs(fabsf(v[s][0].x), v[s][0].y, v[s][1].x), fabsf(v[s][1].y));
        };
        auto pair_max = [&](int m) {     // magnitude maximum of the lane's eight values of slots 2m, 2m+1
            float a = max3abs(fabsf(v[2 * m][0].x), v[2 * m][0].y, v[2 * m][1].x);
            a = max3abs(a, v[2 * m][1].y, v[2 * m + 1][0].x);
            a = max3abs(a, v[2 * m + 1][0].y, v[2 * m + 1][1].x);
            return fmaxf(a, fabsf(v[2 * m + 1][1].y));
        };
        if (MODE == MODE_G128) slot_maxima();

        const uint32_t code_buf = code_base + par2 * SEG_CODE_BYTES;
        const uint32_t code_addr0 = code_buf + code_lane;
        uint8_t *code_gen = fsmem + FastSmem::codes + (size_t)warp * (2 * SEG_CODE_BYTES) + (size_t)par2 * SEG_CODE_BYTES;
        bulk_store_wait_read<1>();           // the store that last read this staging buffer has drained
        __syncwarp();

        if (MODE == MODE_ASYM) {
            // ---------------------------------------------------------------- asymmetric INT4 per token
            // step s = (max y - min y) / 15, zero point z = rne(min y / s), code = clip(rne(y / s) - z, 0, 15).
            // A held value is sgn[class of its slot] times the true output.
            constexpr int CB_ = LOG2B - 4;
            const float INF = __int_as_float(0x7f800000);
            float chi[NCLS], clo[NCLS];
#pragma unroll
            for (int k = 0; k < NCLS; ++k) { chi[k] = -INF; clo[k] = INF; }
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int k = s & 3 & PM;
                chi[k] = fmaxf(fmaxf(chi[k], v[s][0].x), v[s][0].y);
                chi[k] = fmaxf(fmaxf(chi[k], v[s][1].x), v[s][1].y);
                clo[k] = fminf(fminf(clo[k], v[s][0].x), v[s][0].y);
                clo[k] = fminf(fminf(clo[k], v[s][1].x), v[s][1].y);
            }
            float lane_hi = -INF, lane_lo = INF;
#pragma unroll
            for (int k = 0; k < NCLS; ++k) {
                const bool pos = sgn[k] > 0.0f;
                lane_hi = fmaxf(lane_hi, pos ? chi[k] : -clo[k]);
                lane_lo = fminf(lane_lo, pos ? clo[k] : -chi[k]);
            }
            const float hw = warp_max_f32(lane_hi), lw = warp_min_f32(lane_lo);
            const uint32_t pidx = par2 * FAST_WARPS + group;
            float hi_row, lo_row, hm = hw, lm = lw;
            if (G > 1) {
                if (lane == 0) { wmax[par2 * FAST_WARPS + group * G + w_in_g] = hw; wmin[par2 * FAST_WARPS + group * G + w_in_g] = lw; }
                named_barrier(1 + group, G * 32);
                hm = (lane < G) ? wmax[par2 * FAST_WARPS + group * G + lane] : -INF;
                lm = (lane < G) ? wmin[par2 * FAST_WARPS + group * G + lane] : INF;
                hi_row = warp_max_f32(hm);
                lo_row = warp_min_f32(lm);
                refill();
            } else {
                hi_row = hw;
                lo_row = lw;
            }
            const float amax = fmaxf(fabsf(hi_row), fabsf(lo_row));
            const bool live = hi_row > lo_row;               // else: every rotated value is the same (a zero row)
            const float e_abs = 2.0f * err_rel * amax + amax * 2.4e-7f;
            const float thr_hi = hi_row - e_abs, thr_lo = lo_row + e_abs;
            const unsigned cand_hi = (G > 1) ? __ballot_sync(0xffffffffu, live && (lane < G) && hm >= thr_hi) : (live ? 1u : 0u);
            const unsigned cand_lo = (G > 1) ? __ballot_sync(0xffffffffu, live && (lane < G) && lm <= thr_lo) : (live ? 1u : 0u);
            const unsigned candw = cand_hi | cand_lo;
            const bool is_cand = (candw >> w_in_g) & 1u;
            const int ncand = __popc(candw);
            if (!live && leader) {
                reinterpret_cast<float *>(p.out_scales)[2 * (size_t)unit] = 0.0f;
                reinterpret_cast<float *>(p.out_scales)[2 * (size_t)unit + 1] = 0.0f;
            }

            // ---- the exact extremes.  Common case: one warp holds the row's candidates for the maximum and one
            // (maybe the same) those for the minimum, each in one slot: the positions are published and
            // recorded, and (s, z) are derived later, 32 rows at a time.  A side with several slots publishes
            // its exact value instead; a row with several candidate warps on a side combines exact values of
            // all of them through the shared accumulators.
            const bool one_each = __popc(cand_hi) == 1 && __popc(cand_lo) == 1;
            // an entry for one side from this warp: the position of its one candidate slot, or the exact key
            auto side_entry = [&](bool hi_side, bool may_be_position) -> unsigned long long {
                uint32_t slot_mask = 0u;
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    const int k = s & 3 & PM;
                    const bool pos = sgn[k] > 0.0f;
                    float t;                                  // the slot's true maximum (hi side) or minimum
                    if (hi_side == pos) {
                        const float hs = fmaxf(fmaxf(v[s][0].x, v[s][0].y), fmaxf(v[s][1].x, v[s][1].y));
                        t = hi_side ? hs : -hs;
                    } else {
                        const float ls = fminf(fminf(v[s][0].x, v[s][0].y), fminf(v[s][1].x, v[s][1].y));
                        t = hi_side ? -ls : ls;
                    }
                    slot_mask |= (hi_side ? (t >= thr_hi) : (t <= thr_lo)) ? (1u << s) : 0u;
                }
                unsigned cw = __ballot_sync(0xffffffffu, slot_mask != 0u);
                const int src0 = (cw != 0u) ? __ffs(cw) - 1 : 0;
                const uint32_t sm0 = __shfl_sync(0xffffffffu, slot_mask, src0);
                if (may_be_position && cw != 0u && (cw & (cw - 1)) == 0u && (sm0 & (sm0 - 1)) == 0u) {
                    const int sl = __ffs(sm0) - 1, lg = src0 >> 2;
                    const int pch = lg * 8 + (sl ^ ((lg & 3) & ~PM));
                    return (unsigned long long)(uint32_t)(w_in_g * SEG_ELEMS + pch * 16 + 4 * (src0 & 3));
                }
                double best = hi_side ? -1.7976931348623157e308 : 1.7976931348623157e308;
                while (cw) {
                    const int src = __ffs(cw) - 1;
                    cw &= cw - 1;
                    uint32_t sm = __shfl_sync(0xffffffffu, slot_mask, src);
                    const int lg = src >> 2;
                    while (sm) {
                        const int sl = __ffs(sm) - 1;
                        sm &= sm - 1;
                        const int pch = lg * 8 + (sl ^ ((lg & 3) & ~PM));      // chunk position in the segment
                        const int blk_elem = (pch >> CB_) << LOG2B;
                        const int i0 = pch * 16 - blk_elem + 4 * (src & 3);
                        const double val = exact_coord4<B>(seg + blk_elem, i0, lane);   // outputs i0 .. i0+3, one per lane & 3
                        best = hi_side ? fmax(best, val) : fmin(best, val);
                    }
                }
                return hi_side ? warp_max_u64(order_key(best)) : ~warp_max_u64(~order_key(best));
            };
            if (is_cand) {
                uint32_t last = 0u;
                unsigned long long rec_hi = 0ull, rec_lo = 0ull;
                const bool mine_hi = (cand_hi >> w_in_g) & 1u, mine_lo = (cand_lo >> w_in_g) & 1u;
                if (one_each) {
                    unsigned long long e_hi = 0ull, e_lo = 0ull;
                    if (mine_hi) e_hi = side_entry(true, true);
                    if (mine_lo) e_lo = side_entry(false, true);
                    if (lane == 0) {
                        if (mine_hi) wpub[pidx] = e_hi;
                        if (mine_lo) wpub2[pidx] = e_lo;
                        __threadfence_block();
                        const uint32_t publishers = (cand_hi == cand_lo) ? 1u : 2u;
                        if (atomicAdd(&wcnt[pidx], 1u) == publishers - 1u) {         // both sides are published
                            wcnt[pidx] = 0u;
                            __threadfence_block();
                            rec_hi = *reinterpret_cast<volatile unsigned long long *>(&wpub[pidx]);
                            rec_lo = *reinterpret_cast<volatile unsigned long long *>(&wpub2[pidx]);
                            *reinterpret_cast<volatile uint32_t *>(&wflag[pidx]) = it + 1u;
                            last = 1u;
                        }
                    }
                } else {
                    const unsigned long long khi = mine_hi ? side_entry(true, false) : 0ull;
                    const unsigned long long klo = mine_lo ? side_entry(false, false) : ~0ull;
                    if (lane == 0) {
                        atomicMax(&wacc[pidx], khi);
                        atomicMin(&wacc2[pidx], klo);
                        __threadfence_block();
                        if (atomicAdd(&wcnt[pidx], 1u) == (uint32_t)(ncand - 1)) {      // last candidate warp of the row
                            rec_hi = atomicExch(&wacc[pidx], 0ull);
                            rec_lo = atomicExch(&wacc2[pidx], ~0ull);
                            wcnt[pidx] = 0u;
                            wpub[pidx] = rec_hi;
                            wpub2[pidx] = rec_lo;
                            __threadfence_block();
                            *reinterpret_cast<volatile uint32_t *>(&wflag[pidx]) = it + 1u;
                            last = 1u;
                        }
                    }
                }
                if (lane == 0 && last) {
                    wreq[nreq] = rec_hi;
                    wreq2[nreq] = rec_lo;
                    wrequ[nreq] = unit;
                }
                nreq += __shfl_sync(0xffffffffu, last, 0);
                if (nreq == 32u) {
                    serve_asym_requests<LOG2B, PERM>(p, wreq, wreq2, wrequ, nreq, lane);
                    nreq = 0;
                }
            }

            // ---- fp32 step and zero point; where rounding the zero point is a close call, the exact one
            const float rng = hi_row - lo_row;
            const float inv = live ? fminf(__fdividef(15.0f, rng), 3.0e38f) : 0.0f;
            const float ar = live ? fminf(amax * inv * (1.0f / 15.0f), 3.0e38f) : 0.0f;     // |y|max / range >= 1/2
            const float vmin = lo_row * inv;
            float z32 = live ? rintf(vmin) : 0.0f;
            const float wz = 30.0f * err_rel * ar * (1.0f + 2.0f * fabsf(lo_row) * inv * (1.0f / 15.0f)) + (fabsf(vmin) + 1.0f) * 1.0e-6f;
            bool have_exact = false;
            double s_ex = 0.0, z_ex = 0.0;
            auto fetch_exact = [&]() -> bool {            // the row's published (s, z); bounded wait
                uint32_t spin = 0;
                while (ld_volatile_shared_u32(&wflag[pidx]) != it + 1u) {
                    if (++spin >= WAIT_SPIN_LIMIT) return false;
                }
                __threadfence_block();
                unsigned long long khi = *reinterpret_cast<volatile unsigned long long *>(&wpub[pidx]);
                unsigned long long klo = *reinterpret_cast<volatile unsigned long long *>(&wpub2[pidx]);
                // a position: the slot's four outputs from the staged row, lane l holding output (l & 3)
                auto slot_values = [&](uint32_t pos) -> double {
                    const uint32_t blk = (pos >> LOG2B) << LOG2B;
                    return PERM ? exact_coord4_perm<B>(raw_row, ptab + blk, (int)(pos - blk), lane)
                                : exact_coord4<B>(raw_row + blk, (int)(pos - blk), lane);
                };
                if (asym_entry_is_position(khi)) {
                    const double val = slot_values((uint32_t)khi);
                    if (asym_entry_is_position(klo) && klo == khi) klo = ~warp_max_u64(~order_key(val));
                    khi = warp_max_u64(order_key(val));
                }
                if (asym_entry_is_position(klo)) klo = ~warp_max_u64(~order_key(slot_values((uint32_t)klo)));
                asym_step_zero(khi, klo, p.sqrt_b, s_ex, z_ex);
                have_exact = true;
                return true;
            };
            // (a wait that runs out only records the error: the warp must go on to the row's next barrier, or
            // its siblings would be stranded there; the fp32 zero point then stands)
            if (live && !(fabsf(vmin - z32) <= 0.5f - wz)) {
                if (fetch_exact()) z32 = (float)z_ex;
                else if (lane == 0) atomicOr(&g_perq_device_error, 2u);
            }

            // ---- quantise: the magic constant carries -z, so the low nibble of the sum is the code
            const float delta = 36.0f * err_rel * ar + 6.0e-7f;
            f32x2 mul_p[NCLS], mul_m[NCLS];
#pragma unroll
            for (int k = 0; k < NCLS; ++k) {
                const float mp = sgn[k] * inv * (1.0f + delta), mm = sgn[k] * inv * (1.0f - delta);
                mul_p[k] = pack2(mp, mp);
                mul_m[k] = pack2(mm, mm);
            }
            const float magic_z = 12582912.0f - z32;          // 1.5 * 2^23 - z
            const f32x2 magic2 = pack2(magic_z, magic_z);
            uint32_t tie_any = 0u;
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int k = s & 3 & PM;
                const f32x2 tp0 = fma2(v[s][0], mul_p[k], magic2), tp1 = fma2(v[s][1], mul_p[k], magic2);
                const f32x2 tm0 = fma2(v[s][0], mul_m[k], magic2), tm1 = fma2(v[s][1], mul_m[k], magic2);
                const uint32_t pp = ((__float_as_uint(tp1.y) * 16u + __float_as_uint(tp1.x)) * 16u + __float_as_uint(tp0.y)) * 16u
                                    + __float_as_uint(tp0.x);
                const uint32_t pm = ((__float_as_uint(tm1.y) * 16u + __float_as_uint(tm1.x)) * 16u + __float_as_uint(tm0.y)) * 16u
                                    + __float_as_uint(tm0.x);
                tie_any |= (pp ^ pm) ? (1u << s) : 0u;       // (the whole sums: a code outside 0..15 carries upwards)
                sts_code<(3 & ~PM)>(code_addr0, s, pp);
            }

            // ---- slots whose two sums differ: all four codes exactly (a carry may have reached a neighbour)
            if (__any_sync(0xffffffffu, tie_any != 0u)) {
                const bool got_exact = have_exact || fetch_exact();
                if (!got_exact && lane == 0) atomicOr(&g_perq_device_error, 2u);     // the codes stay as staged
                // elements whose two sums differ; all four of a slot in which a sum left 0..15 (its carry
                // may have reached a neighbour)
                uint32_t fm = 0u;
                if (got_exact && tie_any != 0u) {
                    const float t_lo = 12582912.0f, t_hi = 12582927.0f;
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        const int k = s & 3 & PM;
                        const f32x2 tp0 = fma2(v[s][0], mul_p[k], magic2), tp1 = fma2(v[s][1], mul_p[k], magic2);
                        const f32x2 tm0 = fma2(v[s][0], mul_m[k], magic2), tm1 = fma2(v[s][1], mul_m[k], magic2);
                        const float t[4] = {tp0.x, tp0.y, tp1.x, tp1.y}, u[4] = {tm0.x, tm0.y, tm1.x, tm1.y};
                        uint32_t bits = 0u;
                        bool outside = false;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            bits |= (t[j] != u[j]) ? (1u << j) : 0u;
                            outside = outside || t[j] < t_lo || t[j] > t_hi || u[j] < t_lo || u[j] > t_hi;
                        }
                        fm |= (outside ? 0xFu : bits) << (4 * s);
                    }
                }
                __syncwarp();
                unsigned tl = __ballot_sync(0xffffffffu, fm != 0u);
                while (tl) {
                    const int src = __ffs(tl) - 1;
                    tl &= tl - 1;
                    uint32_t fs = __shfl_sync(0xffffffffu, fm, src);
                    while (fs) {
                        const int e = __ffs(fs) - 1;
                        fs &= fs - 1;
                        int blk_elem, i, elem;
                        locate<LOG2B>(src >> 2, src & 3, e, blk_elem, i, elem);
                        const uint16_t *bp;
                        block_of(elem, bp, i);
                        const double ue = exact_coord_fast<BF>(bp, i, lane);
                        if (lane == 0) {
                            uint32_t code = 0u;
                            if (s_ex != 0.0) {
                                const double qd = rint(over_sqrt_b(ue) / s_ex) - z_ex;
                                code = (uint32_t)((int)fmin(fmax(qd, 0.0), 15.0));
                            }
                            uint8_t *cp = code_gen + (elem >> 1);
                            *cp = (elem & 1) ? (uint8_t)((*cp & 0x0F) | (code << 4)) : (uint8_t)((*cp & 0xF0) | code);
                        }
                        __syncwarp();
                    }
                }
            }
        } else if (MODE != MODE_MX) {
            // lane maximum, then the maximum of the scale range in fp32 (a32); the exact maximum
            // (a_bits, bit pattern of a double) only where it is known without waiting
            const float lane_max = (MODE == MODE_G128)
                ? fmaxf(fmaxf(fmaxf(ms[0], ms[1]), fmaxf(ms[2], ms[3])), fmaxf(fmaxf(ms[4], ms[5]), fmaxf(ms[6], ms[7])))
                : fmaxf(fmaxf(pair_max(0), pair_max(1)), fmaxf(pair_max(2), pair_max(3)));
            float a32;
            unsigned long long a_bits = 0ull;
            bool have_exact = true;          // warp-uniform: a_bits is the range's exact maximum
            bool is_cand = false;            // per token: this warp holds candidates for the row maximum
            uint32_t my_pos = 0xffffffffu;   // common case: position of the one slot that holds the range's maximum
            int ncand = 1;
            const uint32_t pidx = par2 * FAST_WARPS + group;
            if (MODE == MODE_G128) {
                // a scale range is the 128 elements of one quad.  Common case: one slot of one lane
                // reaches the threshold; its position is recorded and the scale stored later.
                a32 = fmaxf(lane_max, __shfl_xor_sync(0xffffffffu, lane_max, 1));
                a32 = fmaxf(a32, __shfl_xor_sync(0xffffffffu, a32, 2));
                const float thr = a32 * (1.0f - 2.0f * err_rel - 2.4e-7f);
                uint32_t slot_mask = 0u;
#pragma unroll
                for (int s = 0; s < 8; ++s) slot_mask |= (ms[s] >= thr) ? (1u << s) : 0u;
                if (!(a32 > 0.0f)) slot_mask = 0u;
                const unsigned cl4 = (__ballot_sync(0xffffffffu, slot_mask != 0u) >> (lane & 28)) & 0xFu;
                const int srcq = (lane & 28) | ((__ffs(cl4) - 1) & 3);
                const uint32_t smq = __shfl_sync(0xffffffffu, slot_mask, srcq);
                // (deferring pays while a block is short and the row can be re-read contiguously)
                constexpr bool DEFER = !PERM && !SWIGLU && LOG2B <= 5;
                const bool simple = DEFER && cl4 != 0u && (cl4 & (cl4 - 1)) == 0u && (smq & (smq - 1)) == 0u;
                if (simple) {
                    const int sl = __ffs(smq) - 1;
                    const int pch = g * 8 + (sl ^ (f_g & ~PM));
                    my_pos = (uint32_t)(pch * 16 + 4 * (srcq & 3));
                }
                const unsigned enq = __ballot_sync(0xffffffffu, simple && q == 0);
                if (simple && q == 0)
                    wreq[nreq + __popc(enq & ((1u << lane) - 1u))] = ((unsigned long long)seg_index << 32) | my_pos;
                nreq += __popc(enq);
                if (!(a32 > 0.0f) && q == 0) reinterpret_cast<float *>(p.out_scales)[seg_index * 8 + g] = 0.0f;
                // rare: several candidates in a quad are evaluated now, by the quad
                const bool has_cand = !simple && (a32 > 0.0f) && (lane_max >= thr);
                unsigned cq = __ballot_sync(0xffffffffu, has_cand) & qmask;
                if (__any_sync(0xffffffffu, cq != 0u)) {
                    double a_exact = 0.0;
                    while (cq) {
                        const int src = __ffs(cq) - 1;
                        cq &= cq - 1;
                        uint32_t cm = 0u;
                        if (lane == src) cm = candidate_mask(v, ms, thr);
                        cm = __shfl_sync(qmask, cm, src);
                        while (cm) {
                            const int e = __ffs(cm) - 1;
                            cm &= cm - 1;
                            int blk_elem, i, elem;
                            locate<LOG2B>(src >> 2, src & 3, e, blk_elem, i, elem);
                            a_exact = fmax(a_exact, fabs(exact_coord_quad<LOG2B>(seg + blk_elem, i, q, qmask)));
                        }
                    }
                    if (has_cand || (!simple && (a32 > 0.0f))) {
                        if (q == 0)
                            reinterpret_cast<float *>(p.out_scales)[seg_index * 8 + g] =
                                (a_exact == 0.0) ? 0.0f : (float)(a_exact * p.inv_7_sqrt_b);
                        a_bits = (unsigned long long)__double_as_longlong(a_exact);
                    }
                }
                if (nreq > 24u) {
                    serve_scale_requests<LOG2BF, MODE, PERM>(p, wreq, nreq, lane);
                    nreq = 0;
                }
            } else {
                const float aw = warp_max_f32(lane_max);
                unsigned candw;
                if (G > 1) {
                    if (lane == 0) wmax[par2 * FAST_WARPS + group * G + w_in_g] = aw;
                    named_barrier(1 + group, G * 32);
                    const float am = (lane < G) ? wmax[par2 * FAST_WARPS + group * G + lane] : 0.0f;
                    a32 = warp_max_f32(am);
                    const float thr_row = a32 * (1.0f - 2.0f * err_rel - 2.4e-7f);
                    candw = __ballot_sync(0xffffffffu, (lane < G) && (a32 > 0.0f) && (am >= thr_row));
                    if (WBITS == 0) refill();
                } else {
                    a32 = aw;
                    candw = (a32 > 0.0f) ? 1u : 0u;
                }
                is_cand = (candw >> w_in_g) & 1u;
                ncand = __popc(candw);
                have_exact = (ncand == 0);
                if (ncand == 0 && leader) reinterpret_cast<float *>(p.out_scales)[unit] = 0.0f;
            }

            // ---- per token: the exact row maximum and the stored scale, by the candidate warps only
            // (before the quantiser, while the rotated values are live anyway: placed after it, the block kept all of
            // them in registers through the quantiser's loop)
            if (TOK && is_cand) {
                const float thr_row = a32 * (1.0f - 2.0f * err_rel - 2.4e-7f);
                slot_maxima();
                uint32_t slot_mask = 0u;
#pragma unroll
                for (int s = 0; s < 8; ++s) slot_mask |= (ms[s] >= thr_row) ? (1u << s) : 0u;
                const unsigned cl = __ballot_sync(0xffffffffu, slot_mask != 0u);
                const int src = __ffs(cl) - 1;
                const uint32_t sm = __shfl_sync(0xffffffffu, slot_mask, src);
                if (!SWIGLU && ncand == 1 && (cl & (cl - 1)) == 0u && (sm & (sm - 1)) == 0u) {
                    // one slot holds the maximum: record it, the scale is stored later
                    const int sl = __ffs(sm) - 1, sg = src >> 2;
                    const int pch = sg * 8 + (sl ^ ((sg & 3) & ~PM));
                    my_pos = (uint32_t)(w_in_g * SEG_ELEMS + pch * 16 + 4 * (src & 3));
                    if (lane == 0) {
                        wreq[nreq] = ((unsigned long long)(unit * (uint32_t)G) << 32) | my_pos;
                        if (G > 1) {
                            wpub[pidx] = (1ull << 63) | my_pos;
                            __threadfence_block();
                            *reinterpret_cast<volatile uint32_t *>(&wflag[pidx]) = it + 1u;
                        }
                    }
                    if (++nreq == 32u) {
                        serve_scale_requests<LOG2BF, MODE, PERM>(p, wreq, nreq, lane);
                        nreq = 0;
                    }
                } else {
                    // several candidates: exact values now, combined over the candidate warps
                    const unsigned long long wb = FULLV
                        ? exact_max_of_candidates<LOG2B, FULLV ? LOG2BF : 0>(raw_row, w_in_g * SEG_ELEMS, ms, thr_row, lane)
                        : exact_max_of_candidates<LOG2B, 0>(seg, 0, ms, thr_row, lane);
                    if (ncand == 1) {
                        a_bits = wb;
                        have_exact = true;
                        if (lane == 0) {
                            reinterpret_cast<float *>(p.out_scales)[unit] =
                                (wb == 0ull) ? 0.0f : (float)(__longlong_as_double((long long)wb) * p.inv_7_sqrt_b);
                            if (G > 1) {
                                wpub[pidx] = wb;
                                __threadfence_block();
                                *reinterpret_cast<volatile uint32_t *>(&wflag[pidx]) = it + 1u;
                            }
                        }
                    } else if (lane == 0) {
                        atomicMax(&wacc[pidx], wb);
                        __threadfence_block();
                        if (atomicAdd(&wcnt[pidx], 1u) == (uint32_t)(ncand - 1)) {      // last candidate warp of the row
                            const unsigned long long fin = atomicExch(&wacc[pidx], 0ull);
                            wcnt[pidx] = 0u;
                            reinterpret_cast<float *>(p.out_scales)[unit] =
                                (fin == 0ull) ? 0.0f : (float)(__longlong_as_double((long long)fin) * p.inv_7_sqrt_b);
                            wpub[pidx] = fin;
                            __threadfence_block();
                            *reinterpret_cast<volatile uint32_t *>(&wflag[pidx]) = it + 1u;
                        }
                    }
                }
            }

            // ---- quantise: packed fp32 multiply-add against the magic constant, with the multiplier
            // nudged up and down by the error bound; elements whose two codes differ are resolved exactly
            const float inv = (a32 > 0.0f) ? fminf(__fdividef(7.0f, a32), 3.0e38f) : 0.0f;
            f32x2 mul_p[NCLS], mul_m[NCLS];
#pragma unroll
            for (int k = 0; k < NCLS; ++k) {
                const float mp = inv * q_cp[k], mm = inv * q_cm[k];
                mul_p[k] = pack2(mp, mp);
                mul_m[k] = pack2(mm, mm);
            }
            const f32x2 magic2 = pack2(MAGIC, MAGIC);
            uint32_t tie_any = 0u;
            uint32_t xw[MODE == MODE_FP4 ? 8 : 1];     // FP4: per slot, the XOR of the two code words (kept for the fix-up)
            // E2M1 elements: the value scaled to [-7, 7] plus / minus an additive window, converted twice
            const float tau = (a32 > 0.0f) ? 8.0f * err_rel + 4.0e-6f : 0.0f;
            const f32x2 tau_p2 = pack2(tau, tau), tau_m2 = pack2(0.0f - tau, 0.0f - tau);     // (+0 for a zero row)
            f32x2 mul_c[NCLS];
#pragma unroll
            for (int k = 0; k < NCLS; ++k) mul_c[k] = pack2(qsgn(k) * inv, qsgn(k) * inv);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int k = s & 3 & PM;
                if (MODE == MODE_FP4) {
                    const f32x2 up0 = fma2(v[s][0], mul_c[k], tau_p2), up1 = fma2(v[s][1], mul_c[k], tau_p2);
                    const f32x2 dn0 = fma2(v[s][0], mul_c[k], tau_m2), dn1 = fma2(v[s][1], mul_c[k], tau_m2);
                    const uint32_t pu = cvt_e2m1x4(up0.x, up0.y, up1.x, up1.y);
                    const uint32_t pd = cvt_e2m1x4(dn0.x, dn0.y, dn1.x, dn1.y);
                    xw[MODE == MODE_FP4 ? s : 0] = pu ^ pd;
                    tie_any |= pu ^ pd;
                    sts_code<(3 & ~PM)>(code_addr0, s, pu);
                    continue;
                }
                const f32x2 tp0 = fma2(v[s][0], mul_p[k], magic2), tp1 = fma2(v[s][1], mul_p[k], magic2);
                const f32x2 tm0 = fma2(v[s][0], mul_m[k], magic2), tm1 = fma2(v[s][1], mul_m[k], magic2);
                const uint32_t pp = ((__float_as_uint(tp1.y) * 16u + __float_as_uint(tp1.x)) * 16u + __float_as_uint(tp0.y)) * 16u
                                    + __float_as_uint(tp0.x);
                const uint32_t pm = ((__float_as_uint(tm1.y) * 16u + __float_as_uint(tm1.x)) * 16u + __float_as_uint(tm0.y)) * 16u
                                    + __float_as_uint(tm0.x);
                tie_any |= pp ^ pm;          // low 16 bits: the four codes (offset by 8) under either multiplier
                sts_code<(3 & ~PM)>(code_addr0, s, pp ^ 0x8888u);
            }
            tie_any &= 0xffffu;

            // ---- exact resolution of near ties (rare)
            if (__any_sync(0xffffffffu, tie_any != 0u)) {
                // flagged elements; FP4: from the kept difference words, and zm marks those whose two codes differ
                // in the sign alone (both magnitudes are zero: they need the sign of the exact value, not the scale
                // and none of its fp64 divisions)
                uint32_t fm = 0u, zm = 0u;
                // The rotated values are formed again from the staged segment: had this rare path used the
                // quantiser's, they would stay in registers until here in every iteration.  (Blocks that span
                // lanes or warps cannot be redone by one warp on its own: those variants keep the values.)
                f32x2 vr[8][2];
                if (!FULLV) {
                    h16_tensor(vr);
                    slot_stages(vr);
                }
                f32x2 (&vq)[8][2] = FULLV ? v : vr;
                if (tie_any != 0u) {
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        const int k = s & 3 & PM;
                        if (MODE == MODE_FP4) {
                            const uint32_t x = xw[MODE == MODE_FP4 ? s : 0];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint32_t xn = (x >> (4 * j)) & 0xFu;
                                fm |= xn ? (1u << (4 * s + j)) : 0u;
                                zm |= (xn == 8u) ? (1u << (4 * s + j)) : 0u;
                            }
                            continue;
                        }
                        const f32x2 tp0 = fma2(vq[s][0], mul_p[k], magic2), tp1 = fma2(vq[s][1], mul_p[k], magic2);
                        const f32x2 tm0 = fma2(vq[s][0], mul_m[k], magic2), tm1 = fma2(vq[s][1], mul_m[k], magic2);
                        const float t[4] = {tp0.x, tp0.y, tp1.x, tp1.y}, u[4] = {tm0.x, tm0.y, tm1.x, tm1.y};
#pragma unroll
                        for (int j = 0; j < 4; ++j) fm |= (t[j] != u[j]) ? (1u << (4 * s + j)) : 0u;
                    }
                }
                const bool need_scale = (MODE != MODE_FP4) || __any_sync(0xffffffffu, (fm & ~zm) != 0u);
                if (!have_exact && need_scale) {
                    unsigned long long d = (1ull << 63) | my_pos;
                    if (my_pos == 0xffffffffu) {      // published by a candidate warp of the row: wait for it
                        uint32_t spin = 0;
                        bool gave_up = false;
                        while (ld_volatile_shared_u32(&wflag[pidx]) != it + 1u) {
                            if (++spin >= WAIT_SPIN_LIMIT) { gave_up = true; break; }
                        }
                        if (gave_up) {
                            // the codes stay as staged; the warp goes on (leaving would strand its siblings at the
                            // row's next barrier)
                            if (lane == 0) atomicOr(&g_perq_device_error, 2u);
                            fm = 0u;
                        }
                        __threadfence_block();
                        d = *reinterpret_cast<volatile unsigned long long *>(&wpub[pidx]);
                    }
                    if (d >> 63) {                    // a position: evaluate its four outputs from the staged row
                        const uint32_t pos = (uint32_t)d & 0xffffu;
                        const uint32_t blk = (pos >> LOG2BF) << LOG2BF;
                        const double val = PERM ? fabs(exact_coord4_perm<BF>(raw_row, ptab + blk, (int)(pos - blk), lane))
                                                : fabs(exact_coord4<BF>(raw_row + blk, (int)(pos - blk), lane));
                        a_bits = warp_max_u64((unsigned long long)__double_as_longlong(val));
                    } else {
                        a_bits = d;
                    }
                }
                __syncwarp();
                unsigned tl = __ballot_sync(0xffffffffu, fm != 0u);
                while (tl) {
                    const int src = __ffs(tl) - 1;
                    tl &= tl - 1;
                    uint32_t fs = __shfl_sync(0xffffffffu, fm, src);
                    const uint32_t zs = __shfl_sync(0xffffffffu, zm, src);
                    // the same sequence of fp64 operations as the definition, so exact ties land on exact halves
                    unsigned long long ab_src = __shfl_sync(0xffffffffu, a_bits, src);
                    if (MODE == MODE_G128) {
                        const uint32_t pos_src = __shfl_sync(0xffffffffu, my_pos, src);
                        if (pos_src != 0xffffffffu) {
                            const uint32_t blk = (pos_src >> LOG2B) << LOG2B;
                            const double val = fabs(exact_coord4<B>(seg + blk, (int)(pos_src - blk), lane));
                            ab_src = warp_max_u64((unsigned long long)__double_as_longlong(val));
                        }
                    }
                    const double a_src = __longlong_as_double((long long)ab_src);
                    // (sign-only fix-ups do not use the scale: spare them its two fp64 divisions)
                    // (symmetric INT4 decides most elements without it, see below)
                    const bool want_s = (MODE == MODE_FP4) ? (fs & ~zs) != 0u : false;
                    double s_src = want_s ? over_sqrt_b(a_src) / 7.0 : 0.0;
                    bool have_s = want_s;
                    while (fs) {
                        const int e = __ffs(fs) - 1;
                        fs &= fs - 1;
                        int blk_elem, i, elem;
                        locate<LOG2B>(src >> 2, src & 3, e, blk_elem, i, elem);
                        const uint16_t *bp;
                        block_of(elem, bp, i);
                        const double ue = exact_coord_fast<BF>(bp, i, lane);
                        if (lane == 0) {
                            uint32_t code = 0u;
                            if (MODE == MODE_FP4 && ((zs >> e) & 1u)) {
                                code = signbit(ue) ? 8u : 0u;          // magnitude zero either way: the sign of y = u / sqrt(b)
                            } else if (MODE == MODE_FP4) {
                                const double y = over_sqrt_b(ue);
                                code = e2m1_code_exact((s_src != 0.0) ? y / s_src : 0.0, signbit(y));
                            } else if (a_src != 0.0) {
                                // The staged code kp comes from the multiplier nudged away from zero, the other
                                // candidate is one step towards zero, the tie between them at |y / s| = |kp| - 1/2.
                                // y / s = 7 u / a: the side is the sign of 14 |u| - (2 |kp| - 1) a, two fp64
                                // products whose rounding errors are far below the margin asked for here.  Only
                                // an exact or all but exact tie takes the definition's own sequence of operations
                                // (three fp64 divisions), which then lands on exact halves where the definition does.
                                const uint32_t nib = (code_gen[elem >> 1] >> ((elem & 1) * 4)) & 0xFu;
                                const int kp = (int)(nib ^ 8u) - 8;
                                const int mag = kp < 0 ? -kp : kp;
                                const double diff = 14.0 * fabs(ue) - (double)(2 * mag - 1) * a_src;
                                if (mag >= 1 && fabs(diff) > a_src * 1.0e-12) {
                                    code = (uint32_t)(diff > 0.0 ? kp : (kp < 0 ? kp + 1 : kp - 1)) & 0xFu;
                                } else {
                                    if (!have_s) { s_src = over_sqrt_b(a_src) / 7.0; have_s = true; }
                                    double qd = rint(over_sqrt_b(ue) / s_src);
                                    qd = fmin(fmax(qd, -8.0), 7.0);
                                    code = (uint32_t)((int)qd) & 0xFu;
                                }
                            }
                            uint8_t *bp = code_gen + (elem >> 1);
                            *bp = (elem & 1) ? (uint8_t)((*bp & 0x0F) | (code << 4)) : (uint8_t)((*bp & 0xF0) | code);
                        }
                        __syncwarp();
                    }
                }
            }
        } else {   // ---------------------------------------------------------------- MXFP4
            // A group of 32 = slots 2m, 2m+1 of the four lanes of a quad.  Lane q of the quad derives
            // the shared exponent of slot pair m = q, then the quad exchanges multipliers.
            float a32, bref;
            {
                const float g0 = pair_max(0), g1 = pair_max(1), g2 = pair_max(2), g3 = pair_max(3);
                const bool q1 = (q & 1) != 0, q2 = (q & 2) != 0;
                float k0 = q2 ? g2 : g0, k1 = q2 ? g3 : g1;
                const float s0 = q2 ? g0 : g2, s1 = q2 ? g1 : g3;
                k0 = fmaxf(k0, __shfl_xor_sync(0xffffffffu, s0, 2));
                k1 = fmaxf(k1, __shfl_xor_sync(0xffffffffu, s1, 2));
                const float keep = q1 ? k1 : k0, send = q1 ? k0 : k1;
                a32 = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, 1));
                // error reference: the largest |u| of the Hadamard block (it may span several groups)
                bref = a32;
                if (CB >= 2) bref = fmaxf(bref, __shfl_xor_sync(0xffffffffu, bref, 1));
                if (CB >= 3) bref = fmaxf(bref, __shfl_xor_sync(0xffffffffu, bref, 2));
                if (FULLV) {     // longer blocks: over their lane groups, then (whole rows) over the row's warps
#pragma unroll
                    for (int bit = 4; bit < (4 << LBITS); bit <<= 1) bref = fmaxf(bref, __shfl_xor_sync(0xffffffffu, bref, bit));
                    if (WBITS > 0) {
                        if (lane == 0) wmax[par2 * FAST_WARPS + warp] = bref;
                        named_barrier(1 + group, G * 32);      // also: every warp has read the exchange space
                        bref = warp_max_f32((lane < G) ? wmax[par2 * FAST_WARPS + group * G + lane] : 0.0f);
                    }
                }
            }
            // E + 127 with E = floor(log2(a / sqrt(b))) - 2, from the bits of a32; near a boundary of
            // that floor the maximum is re-derived exactly
            const uint32_t bits = __float_as_uint(a32);
            const int e8 = (int)(bits >> 23);
            int Eb;
            float dist;
            if ((LOG2BF & 1) == 0) {
                Eb = e8 - LOG2BF / 2 - 2;
                const float lower = __uint_as_float(bits & 0x7f800000u);
                dist = fminf(a32 - lower, 2.0f * lower - a32);
            } else {
                const uint32_t mant = bits & 0x7fffffu;
                Eb = e8 - (LOG2BF - 1) / 2 - 3 + (mant >= 0x3504f4u ? 1 : 0);
                dist = fabsf(a32 - __uint_as_float((bits & 0x7f800000u) | 0x3504f3u));
            }
            const float tol = 2.0f * err_rel * bref + a32 * 2.4e-7f;
            const bool near = (a32 > 0.0f) && (dist <= tol || e8 == 0);
            const unsigned near_w = __ballot_sync(0xffffffffu, near);
            if (FULLV && near_w != 0u) {   // rare; whole-row blocks are evaluated by the whole warp, one group at a time
                unsigned nw = near_w;
                while (nw) {
                    const int owner = __ffs(nw) - 1;
                    nw &= nw - 1;
                    const int m = owner & 3;
                    const float thr = __shfl_sync(0xffffffffu, a32 - tol, owner);
                    uint32_t mymask = 0u;
                    if ((lane >> 2) == (owner >> 2)) {
#pragma unroll
                        for (int mm = 0; mm < 4; ++mm) {
                            if (mm == m) {
                                const float e[8] = {v[2 * mm][0].x, v[2 * mm][0].y, v[2 * mm][1].x, v[2 * mm][1].y,
                                                    v[2 * mm + 1][0].x, v[2 * mm + 1][0].y, v[2 * mm + 1][1].x, v[2 * mm + 1][1].y};
#pragma unroll
                                for (int k = 0; k < 8; ++k) mymask |= (fabsf(e[k]) >= thr) ? (1u << k) : 0u;
                            }
                        }
                    }
                    double best = 0.0;
                    for (int ql = 0; ql < 4; ++ql) {
                        uint32_t cm = __shfl_sync(0xffffffffu, mymask, (owner & 28) | ql);
                        while (cm) {
                            const int k = __ffs(cm) - 1;
                            cm &= cm - 1;
                            int blk_elem, i, elem;
                            locate<LOG2B>(owner >> 2, ql, 8 * m + k, blk_elem, i, elem);
                            const uint16_t *bp;
                            block_of(elem, bp, i);
                            best = fmax(best, fabs(exact_coord_fast<BF>(bp, i, lane)));
                        }
                    }
                    if (lane == owner) {
                        int ex;
                        (void)frexp(over_sqrt_b(best), &ex);
                        Eb = ex - 3 + 127;
                    }
                }
            } else if (near_w != 0u) {   // rare: exact maximum of the group from every element that could attain it
                const unsigned nearq = (near_w >> (lane & 28)) & 0xFu;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    if ((nearq >> m) & 1u) {
                        const int owner = (lane & 28) | m;
                        const float a_m = __shfl_sync(qmask, a32, owner), tol_m = __shfl_sync(qmask, tol, owner);
                        const float thr = a_m - tol_m;
                        const bool has = pair_max(m) >= thr;
                        unsigned cq = __ballot_sync(qmask, has) & qmask;
                        double best = 0.0;
                        while (cq) {
                            const int src = __ffs(cq) - 1;
                            cq &= cq - 1;
                            uint32_t cm = 0u;
                            if (lane == src) {
                                const float e[8] = {v[2 * m][0].x, v[2 * m][0].y, v[2 * m][1].x, v[2 * m][1].y,
                                                    v[2 * m + 1][0].x, v[2 * m + 1][0].y, v[2 * m + 1][1].x, v[2 * m + 1][1].y};
#pragma unroll
                                for (int k = 0; k < 8; ++k) cm |= (fabsf(e[k]) >= thr) ? (1u << k) : 0u;
                            }
                            cm = __shfl_sync(qmask, cm, src);
                            while (cm) {
                                const int k = __ffs(cm) - 1;
                                cm &= cm - 1;
                                int blk_elem, i, elem;
                                locate<LOG2B>(src >> 2, src & 3, 8 * m + k, blk_elem, i, elem);
                                best = fmax(best, fabs(exact_coord_quad<LOG2B>(seg + blk_elem, i, q, qmask)));
                            }
                        }
                        if (q == m) {
                            int ex;
                            (void)frexp(over_sqrt_b(best), &ex);
                            Eb = ex - 3 + 127;
                        }
                    }
                }
            }
            Eb = min(max(Eb, 0), 254);
            // multiplier 2^-E / sqrt(b) and the additive rounding window, in scaled units
            float c;
            if ((LOG2BF & 1) == 0) c = __uint_as_float((uint32_t)min(max(254 - Eb - LOG2BF / 2, 1), 254) << 23);
            else c = __uint_as_float((uint32_t)min(max(254 - Eb - (LOG2BF - 1) / 2, 1), 254) << 23) * 0.70710678118654752f;
            uint32_t byte = (uint32_t)Eb;
            if (!(a32 > 0.0f)) { c = 0.0f; byte = 0u; }
            // (an all-zero block is exact: no window, so that its zeros are not flagged for their sign)
            const float tau = (bref > 0.0f) ? 2.0f * err_rel * bref * c + 2.0e-6f : 0.0f;
            // scale bytes of the quad's four groups: slot pair m is chunk pair m ^ (f >> 1)
            uint32_t word = byte << (8 * (q ^ ((f_g & ~PM) >> 1)));
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            if (q == 0) reinterpret_cast<uint32_t *>(p.out_scales)[seg_index * 8 + g] = word;

            uint32_t tie_any = 0u;
            f32x2 mulc[8], tau_p[4], tau_m[4];
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const float c_m = __shfl_sync(0xffffffffu, c, (lane & 28) | m);
                const float t_m = __shfl_sync(0xffffffffu, tau, (lane & 28) | m);
                tau_p[m] = pack2(t_m, t_m);
                tau_m[m] = pack2(0.0f - t_m, 0.0f - t_m);   // +0 for a zero window: (-0) + (+0) = +0 on both sides
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float mc = qsgn((2 * m + h) & 3 & PM) * c_m;
                    mulc[2 * m + h] = pack2(mc, mc);
                }
            }
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const f32x2 up0 = fma2(v[s][0], mulc[s], tau_p[s >> 1]), up1 = fma2(v[s][1], mulc[s], tau_p[s >> 1]);
                const f32x2 dn0 = fma2(v[s][0], mulc[s], tau_m[s >> 1]), dn1 = fma2(v[s][1], mulc[s], tau_m[s >> 1]);
                const uint32_t pu = cvt_e2m1x4(up0.x, up0.y, up1.x, up1.y);
                const uint32_t pd = cvt_e2m1x4(dn0.x, dn0.y, dn1.x, dn1.y);
                tie_any |= pu ^ pd;
                sts_code<(3 & ~PM)>(code_addr0, s, pu);
            }
            if (__any_sync(0xffffffffu, tie_any != 0u)) {
                uint32_t fm = 0u;
                if (tie_any != 0u) {
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        const f32x2 up0 = fma2(v[s][0], mulc[s], tau_p[s >> 1]), up1 = fma2(v[s][1], mulc[s], tau_p[s >> 1]);
                        const f32x2 dn0 = fma2(v[s][0], mulc[s], tau_m[s >> 1]), dn1 = fma2(v[s][1], mulc[s], tau_m[s >> 1]);
                        const uint32_t x0 = cvt_e2m1x2(up0.x, up0.y) ^ cvt_e2m1x2(dn0.x, dn0.y);
                        const uint32_t x1 = cvt_e2m1x2(up1.x, up1.y) ^ cvt_e2m1x2(dn1.x, dn1.y);
                        fm |= ((x0 & 0x0Fu) ? 1u : 0u) << (4 * s) | ((x0 & 0xF0u) ? 2u : 0u) << (4 * s);
                        fm |= ((x1 & 0x0Fu) ? 4u : 0u) << (4 * s) | ((x1 & 0xF0u) ? 8u : 0u) << (4 * s);
                    }
                }
                __syncwarp();
                unsigned tl = __ballot_sync(0xffffffffu, fm != 0u);
                while (tl) {
                    const int src = __ffs(tl) - 1;
                    tl &= tl - 1;
                    uint32_t fs = __shfl_sync(0xffffffffu, fm, src);
                    const uint32_t wsrc = __shfl_sync(0xffffffffu, word, src);
                    const int fsrc = (((src >> 2) & 3) & ~PM) >> 1;
                    while (fs) {
                        const int e = __ffs(fs) - 1;
                        fs &= fs - 1;
                        int blk_elem, i, elem;
                        locate<LOG2B>(src >> 2, src & 3, e, blk_elem, i, elem);
                        const uint16_t *bp;
                        block_of(elem, bp, i);
                        const double ue = exact_coord_fast<BF>(bp, i, lane);
                        if (lane == 0) {
                            const int E = (int)((wsrc >> (8 * ((e >> 3) ^ fsrc))) & 0xFFu) - 127;
                            const double y = over_sqrt_b(ue);
                            const uint32_t code = e2m1_code_exact(scalbn(y, -E), signbit(y));
                            uint8_t *bp = code_gen + (elem >> 1);
                            *bp = (elem & 1) ? (uint8_t)((*bp & 0x0F) | (code << 4)) : (uint8_t)((*bp & 0xF0) | code);
                        }
                        __syncwarp();
                    }
                }
            }
        }

        // ---- packed codes: shared staging -> global
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
            bulk_store(code_out, code_buf, SEG_CODE_BYTES);
            if (PERM) mbar_arrive(empty_base + stage * 8);     // this warp no longer reads the staged row
        }
    }
    if (MODE == MODE_ASYM) {
        if (nreq > 0u) serve_asym_requests<LOG2B, PERM>(p, wreq, wreq2, wrequ, nreq, lane);
    } else if (MODE != MODE_MX && nreq > 0u) {
        serve_scale_requests<LOG2BF, MODE, PERM>(p, wreq, nreq, lane);
    }
    bulk_store_wait_read<0>();
}

}  // namespace perq
