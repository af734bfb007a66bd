// Full-vector rotate+quantize kernel (b = d in {1024, 2048, 4096}, unpermuted), MXFP4 or INT4 per token.
//
// The rotation by H_d is split by index bits.  The low seven bits are the tensor-core kernels' own: H_16 on the
// tensor cores plus three packed stages in registers rotate every 128-element chunk of a warp's 1024-element
// segment (tok_rotate<7>).  The remaining log2(d) - 7 bits pair values that live in different lanes and
// different warps; instead of shuffles and a warp-to-warp exchange (three shuffle stages per element and G
// fp32 copies of every segment through shared memory, which is what bounded the group kernel's b = d variants)
// every value makes ONE round trip through shared memory:
//
//   pass 1   warp w of a row writes its rotated chunks to the row's fp32 tile Y[chunk][128] (16-byte stores,
//            rows padded to 144 floats: conflict-free), and the row's warps meet at a named barrier;
//   pass 2   a lane reads, for its column(s) j of the tile, the values of ALL d / 128 chunks (consecutive
//            lanes read consecutive words) and runs the remaining butterfly stages on registers: 32 values per
//            lane, packed add/sub.  Sylvester matrices are Kronecker powers of H_2, so rotating the chunk
//            index after the position inside the chunk is the same matrix, natural order.
//   regroup  a warp's outputs are 32 scale groups of 32 consecutive outputs, one VALUE of each per lane; a
//            32 x 32 transpose through the warp's own (by then idle) rows of Y hands every lane one whole
//            group: its maximum, exponent, multiplier, codes and the 16 bytes it stores are lane-local.
//
// Exactness rules, error model (K = 1 for whole rows) and formats as in perq_fast.cuh; the rare paths (a group
// maximum near an exponent boundary, an element whose two conversions differ, the exact row maximum) are
// functions that are not inlined and read the staged bf16 row and the regrouped values again.
#pragma once
#include "perq_mx.cuh"

namespace perq {

constexpr int FULL_NSTAGE = 3;                // ring stages (rows) per group of warps
constexpr int FULL_YS = 144;                  // floats per chunk row of Y: 128 + 16, so that the two lane groups of a
                                              // quarter warp store to different halves of the banks
constexpr int FULL_TS = 36;                   // floats per row of the regrouping tile (32 + 4: 16-byte reads of
                                              // eight lanes fall in distinct bank quads)

// Shared memory relative to a 1024-byte aligned base: 16 warps x 3 stages x 2 KB of bf16 input, 4608 bytes
// of fp32 tile per warp (8 chunk rows of 144 floats = 32 regrouping rows of 36 floats), mbarriers, row maxima.
struct FullSmem {
    static constexpr size_t stages = 0;
    static constexpr size_t tile = stages + (size_t)FAST_WARPS * FULL_NSTAGE * SEG_BYTES;
    static constexpr size_t full = tile + (size_t)FAST_WARPS * 8 * FULL_YS * 4;
    static constexpr size_t xch = full + (size_t)FAST_WARPS * FULL_NSTAGE * 8;       // [2][16] fp32 warp maxima, 8 bytes apart
    static constexpr size_t wreq = xch + (size_t)2 * FAST_WARPS * 8;                 // [16][16] u64 deferred scale records
    static constexpr size_t used = wreq + (size_t)FAST_WARPS * 16 * 8;
    static constexpr size_t total = used + 1024;
};
static_assert(8 * FULL_YS == 32 * FULL_TS, "the regrouping tile reuses the warp's chunk rows");

__device__ __forceinline__ void lds_v2f(uint32_t addr, float &a, float &b)
{
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}
__device__ __forceinline__ float lds_f(uint32_t addr)
{
    float a;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(a) : "r"(addr) : "memory");
    return a;
}
__device__ __forceinline__ void sts_f(uint32_t addr, float a) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(a) : "memory"); }
__device__ __forceinline__ void sts_v2f(uint32_t addr, float a, float b)
{
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}

// A lane's group of 32 regrouped values (row `lane` of the warp's tile).
__device__ __forceinline__ void full_load_group(uint32_t t_lane, f32x2 (&q)[16])
{
#pragma unroll
    for (int c = 0; c < 8; ++c) lds_v4f(t_lane + c * 16, q[2 * c].x, q[2 * c].y, q[2 * c + 1].x, q[2 * c + 1].y);
}

template <int LOG2D>
__device__ __forceinline__ double full_over_sqrt_d(double u, double sqrt_d)
{
    return (LOG2D % 2 == 0) ? u * (1.0 / (double)(1 << (LOG2D / 2))) : u / sqrt_d;
}

// Exact unnormalised output i of the whole-row block, sum_k (-1)^{popcount(i & k)} x_k over the staged bf16 row,
// by one warp: 16-byte loads (a lane takes 8 consecutive inputs of every 256), the signs of a piece from one
// parity of the piece's position and a per-call pattern for its low three bits, four independent fp64
// accumulators per lane.  Every lane returns lane 0's sum (the lanes add in different orders).
template <int LOG2D>
__device__ __forceinline__ double full_exact_coord(const uint16_t *raw_row, uint32_t i, int lane)
{
    constexpr int D = 1 << LOG2D;
    uint32_t flipw[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
        flipw[j] = ((__popc(i & (uint32_t)(2 * j)) & 1) ? 0x8000u : 0u) | ((__popc(i & (uint32_t)(2 * j + 1)) & 1) ? 0x80000000u : 0u);
    const uint4 *src = reinterpret_cast<const uint4 *>(raw_row) + lane;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll 4
    for (int r = 0; r < D / 256; ++r) {
        const uint4 w4 = src[r * 32];
        const uint32_t base = (__popc(i & (uint32_t)(r * 256 + lane * 8)) & 1) ? 0x80008000u : 0u;
        const uint32_t w[4] = {w4.x ^ flipw[0] ^ base, w4.y ^ flipw[1] ^ base, w4.z ^ flipw[2] ^ base, w4.w ^ flipw[3] ^ base};
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] += bf16_bits_to_f64(w[j]) + bf16_bits_to_f64(w[j] >> 16);
    }
    double sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    return __shfl_sync(0xffffffffu, sum, 0);
}

// Rare: the exact shared exponents of the groups whose fp32 maximum is within tol of a value at which the
// exponent changes (near).  Every element of such a group that could attain the maximum is evaluated exactly
// (a d-term fp64 sum over the staged row, by the whole warp); i0 is the row position of the lane's group.
template <int LOG2D>
__device__ __noinline__ int full_mx_exact_exponents(uint32_t t_lane, const uint16_t *raw_row, float a32, float tol, bool near, int Eb,
                                                    uint32_t i0, double sqrt_d, int lane)
{
    f32x2 q[16];
    full_load_group(t_lane, q);
    unsigned nw = __ballot_sync(0xffffffffu, near);
    while (nw) {
        const int owner = __ffs(nw) - 1;
        nw &= nw - 1;
        const float thr = a32 - tol;
        uint32_t cm = 0u;
#pragma unroll
        for (int m = 0; m < 16; ++m) cm |= (fabsf(q[m].x) >= thr ? 1u : 0u) << (2 * m) | (fabsf(q[m].y) >= thr ? 2u : 0u) << (2 * m);
        cm = __shfl_sync(0xffffffffu, cm, owner);
        const uint32_t io = __shfl_sync(0xffffffffu, i0, owner);
        double best = 0.0;
        while (cm) {
            const int k = __ffs(cm) - 1;
            cm &= cm - 1;
            best = fmax(best, fabs(full_exact_coord<LOG2D>(raw_row, io + k, lane)));
        }
        if (lane == owner) {
            int ex;
            (void)frexp(full_over_sqrt_d<LOG2D>(best, sqrt_d), &ex);
            Eb = ex - 3 + 127;
        }
    }
    return Eb;
}

// Rare: exact E2M1 codes of the elements whose two conversions differ.  The lane's values are read again from
// the regrouping tile, the flags are formed again, every flagged element is evaluated exactly by the whole
// warp, and the owning lane rewrites the nibble in the 16 bytes it has already stored.
template <int LOG2D>
__device__ __noinline__ void full_mx_fix_ties(uint32_t t_lane, const uint16_t *raw_row, float c, float tau, int Eb, uint32_t i0,
                                              uint8_t *out16, double sqrt_d, int lane)
{
    f32x2 q[16];
    full_load_group(t_lane, q);
    const f32x2 c2 = pack2(c, c), tp = pack2(tau, tau), tm = pack2(0.0f - tau, 0.0f - tau);
    uint32_t fm = 0u;
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        const f32x2 up = fma2(q[m], c2, tp), dn = fma2(q[m], c2, tm);
        const uint32_t x = cvt_e2m1x2(up.x, up.y) ^ cvt_e2m1x2(dn.x, dn.y);
        fm |= ((x & 0x0Fu) ? 1u : 0u) << (2 * m) | ((x & 0xF0u) ? 2u : 0u) << (2 * m);
    }
    unsigned tl = __ballot_sync(0xffffffffu, fm != 0u);
    while (tl) {
        const int src = __ffs(tl) - 1;
        tl &= tl - 1;
        uint32_t fs = __shfl_sync(0xffffffffu, fm, src);
        const uint32_t io = __shfl_sync(0xffffffffu, i0, src);
        while (fs) {
            const int e = __ffs(fs) - 1;
            fs &= fs - 1;
            const double ue = full_exact_coord<LOG2D>(raw_row, io + e, lane);
            if (lane == src) {
                const double y = full_over_sqrt_d<LOG2D>(ue, sqrt_d);
                const uint32_t code = e2m1_code_exact(scalbn(y, -(Eb - 127)), signbit(y));
                uint8_t *bp = out16 + (e >> 1);
                *bp = (e & 1) ? (uint8_t)((*bp & 0x0F) | (code << 4)) : (uint8_t)((*bp & 0xF0) | code);
            }
        }
    }
}

// MODE_MX only (for now): template parameter kept for the per-token formats.
template <int LOG2D, int MODE>
__global__ void __launch_bounds__(FAST_THREADS, 1) perq_full_kernel(FastParams p)
{
    static_assert(LOG2D >= 10 && LOG2D <= 12, "rows of 1024, 2048 or 4096 channels");
    static_assert(MODE == MODE_MX, "MXFP4");
    constexpr int LOG2W = LOG2D - 10;             // warps per row: one per 1024-element segment
    constexpr int W = 1 << LOG2W;
    constexpr int GROUPS = FAST_WARPS / W;
    constexpr int LOG2R = LOG2D - 7;              // chunk-index bits: values per column
    constexpr int R = 1 << LOG2R;
    constexpr int C = 32 / R;                     // columns per lane (1, 2 or 4): 32 values per lane either way
    constexpr int LOG2C = 5 - LOG2R;
    constexpr int NST = FULL_NSTAGE;
    constexpr uint32_t UNIT_BYTES = (uint32_t)W * SEG_BYTES;
    constexpr uint32_t UNIT_ELEMS = (uint32_t)W * SEG_ELEMS;
    extern __shared__ __align__(128) unsigned char fsmem_raw[];
    unsigned char *fsmem = fsmem_raw + ((1024u - (smem_u32(fsmem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = warp >> LOG2W, w_in_g = warp & (W - 1);
    const int g = lane >> 2, q4 = lane & 3;
    const float err_rel = FAST_ERR_K_FULL * (float)LOG2D * TWO_M24;

    const uint32_t smem_base = smem_u32(fsmem);
    const uint32_t stage_base = smem_base + (uint32_t)FullSmem::stages + (uint32_t)group * (NST * UNIT_BYTES);
    const uint32_t seg_base = stage_base + (uint32_t)w_in_g * SEG_BYTES;
    const uint32_t full_base = smem_base + (uint32_t)FullSmem::full + (uint32_t)group * (NST * 8);
    const uint32_t y_group = smem_base + (uint32_t)FullSmem::tile + (uint32_t)(group * W) * (8 * FULL_YS * 4);   // the row's tile
    const uint32_t y_warp = y_group + (uint32_t)w_in_g * (8 * FULL_YS * 4);                                      // this warp's chunk rows
    const uint32_t xch_group = smem_base + (uint32_t)FullSmem::xch + (uint32_t)(group * W) * 8;

    if (tid < FAST_WARPS * NST) mbar_init(smem_base + (uint32_t)FullSmem::full + tid * 8, 1);
    if (tid == 0) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    griddep_wait();             // nothing above reads or writes global memory
    griddep_launch();

    const uint32_t first = blockIdx.x * GROUPS + group;
    const uint32_t stride = gridDim.x * GROUPS;
    if (first >= p.units_total) return;          // whole groups leave together
    const uint32_t n_units = (p.units_total - first + stride - 1) / stride;
    const uint32_t refill_end = n_units > (uint32_t)NST ? n_units - NST : 0u;
    const bool leader = (w_in_g == 0) && (lane == 0);

    TokLane<7> L;
    L.init(lane);
    f32x2 sg2[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) sg2[k] = pack2(L.sgn[k], L.sgn[k]);

    const size_t unit_step_elems = (size_t)stride * UNIT_ELEMS;
    const uint16_t *xload = p.x + (size_t)first * UNIT_ELEMS;
    if (leader) {
#pragma unroll
        for (int s = 0; s < NST; ++s) {
            if ((uint32_t)s < n_units) {
                mbar_expect_tx(full_base + s * 8, UNIT_BYTES);
                bulk_load(stage_base + s * UNIT_BYTES, xload, UNIT_BYTES, full_base + s * 8);
                xload += unit_step_elems;
            }
        }
    }
    // pass 1: this lane's 16-byte pieces go to chunk row 8 w + g, columns 16 s + 4 q .. + 3
    const uint32_t y_store = y_warp + (uint32_t)(g * FULL_YS + 4 * q4) * 4;
    // pass 2: this lane's C columns of every chunk row
    const uint32_t y_load = y_group + (uint32_t)((w_in_g * 32 + lane) * C) * 4;
    // regrouping tile (this warp's chunk rows again): row `lane` is the lane's group
    const uint32_t t_lane = y_warp + (uint32_t)lane * (FULL_TS * 4);
    // the lane's group: outputs i0 .. i0 + 31 of the row
    const uint32_t i0 = (uint32_t)(lane >> LOG2C) * 128u + 32u * (uint32_t)(C * w_in_g + (lane & (C - 1)));
    uint8_t *outp = p.out_codes + (size_t)first * (UNIT_ELEMS / 2) + i0 / 2;
    const size_t out_step = (size_t)stride * (UNIT_ELEMS / 2);
    uint8_t *scale_out = reinterpret_cast<uint8_t *>(p.out_scales) + (size_t)first * (UNIT_ELEMS / 32) + i0 / 32;
    const size_t scale_step = (size_t)stride * (UNIT_ELEMS / 32);
    const uint16_t *stage_gen = reinterpret_cast<const uint16_t *>(fsmem + FullSmem::stages);

    uint32_t xch_it = xch_group;
    uint32_t stage = 0, parity = 0;
    bool ok = true;
    for (uint32_t it = 0; it < n_units; ++it, outp += out_step, scale_out += scale_step, xch_it ^= FAST_WARPS * 8) {
        const uint32_t bar = full_base + stage * 8;
        if (!mbar_try_once(bar, parity) && !mbar_wait(bar, parity)) { ok = false; break; }
        const uint32_t row_addr = stage_base + stage * UNIT_BYTES;

        // ---- pass 1: H_128 on the segment's eight chunks, true signs, fp32 tile
        {
            f32x2 v[8][2];
            tok_rotate<7>(seg_base + stage * UNIT_BYTES, L, v);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const f32x2 a = mul2(v[s][0], sg2[s & 3]), b = mul2(v[s][1], sg2[s & 3]);
                sts_v4f(y_store + s * 64, a.x, a.y, b.x, b.y);
            }
        }
        if (W > 1) named_barrier(1 + group, W * 32); else __syncwarp();
        // every warp of the row is past the previous iteration: its stage is refilled
        if (w_in_g == 0) {
            const uint32_t ps = stage == 0 ? (uint32_t)(NST - 1) : stage - 1u;
            const bool go = (lane == 0) && (it - 1u < refill_end);
            bulk_load_if(go, stage_base + ps * UNIT_BYTES, xload, UNIT_BYTES, full_base + ps * 8);
            if (go) xload += unit_step_elems;
        }

        // ---- pass 2: the chunk-index bits, on registers
        f32x2 u[16];
        if (C == 1) {
#pragma unroll
            for (int m = 0; m < 16; ++m) { u[m].x = lds_f(y_load + m * (FULL_YS * 4)); u[m].y = lds_f(y_load + (m + 16) * (FULL_YS * 4)); }
        } else if (C == 2) {
#pragma unroll
            for (int k = 0; k < 16; ++k) lds_v2f(y_load + k * (FULL_YS * 4), u[k].x, u[k].y);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) lds_v4f(y_load + k * (FULL_YS * 4), u[2 * k].x, u[2 * k].y, u[2 * k + 1].x, u[2 * k + 1].y);
        }
        {
            // packed stages over the bits of the register index that are chunk-index bits
            constexpr int LO = (C == 4) ? 1 : 0;                 // C == 4: bit 0 of the register index is a column pair
            constexpr int NB = (C == 1) ? 4 : LOG2R;             // C == 1: chunk bit 4 is inside the pair
#pragma unroll
            for (int t = 0; t < NB; ++t) {
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    if ((m & (1 << (t + LO))) == 0) {
                        const f32x2 a = u[m], c2 = u[m | (1 << (t + LO))];
                        u[m] = add2(a, c2);
                        u[m | (1 << (t + LO))] = sub2(a, c2);
                    }
                }
            }
            if (C == 1) {
#pragma unroll
                for (int m = 0; m < 16; ++m) { const float a = u[m].x, b = u[m].y; u[m].x = a + b; u[m].y = a - b; }
            }
        }
        // the row's largest fp32 magnitude: the reference of the error bound (the block is the row)
        float bref;
        {
            float lm = 0.0f;
#pragma unroll
            for (int m = 0; m < 16; ++m) lm = max3abs(lm, u[m].x, u[m].y);
            bref = warp_max_f32(lm);
            if (W > 1) {
                if (lane == 0) asm volatile("st.shared.b32 [%0], %1;" ::"r"(xch_it + (uint32_t)w_in_g * 8), "r"(__float_as_uint(bref)) : "memory");
                named_barrier(1 + group, W * 32);     // also: every warp of the row has read the tile
                uint32_t ob;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(ob) : "r"(xch_it + (uint32_t)(lane & (W - 1)) * 8) : "memory");
                bref = warp_max_f32(__uint_as_float(ob));
            } else {
                __syncwarp();
            }
        }
        // ---- regroup: value (chunk k', column) -> row k' * C + column / 32 of the tile, then one row per lane
        if (C == 1) {
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                sts_f(y_warp + (uint32_t)(m * FULL_TS + lane) * 4, u[m].x);
                sts_f(y_warp + (uint32_t)((m + 16) * FULL_TS + lane) * 4, u[m].y);
            }
        } else if (C == 2) {
#pragma unroll
            for (int k = 0; k < 16; ++k) sts_v2f(y_warp + (uint32_t)((2 * k + (lane >> 4)) * FULL_TS + ((2 * lane) & 31)) * 4, u[k].x, u[k].y);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                sts_v4f(y_warp + (uint32_t)((4 * k + (lane >> 3)) * FULL_TS + ((4 * lane) & 31)) * 4, u[2 * k].x, u[2 * k].y, u[2 * k + 1].x, u[2 * k + 1].y);
        }
        __syncwarp();
        full_load_group(t_lane, u);

        // ---- the lane's scale group: maximum, shared exponent, multiplier, window
        float a32 = 0.0f;
#pragma unroll
        for (int m = 0; m < 16; ++m) a32 = max3abs(a32, u[m].x, u[m].y);
        const uint16_t *raw_row = stage_gen + (row_addr - smem_base - (uint32_t)FullSmem::stages) / 2;
        float dist;
        int Eb = mx_exponent_fp32<LOG2D>(a32, dist);
        const float tol = 2.0f * err_rel * bref + a32 * 2.4e-7f;
        const bool near = (a32 > 0.0f) && (dist <= tol || (__float_as_uint(a32) >> 23) == 0u);
        if (__any_sync(0xffffffffu, near)) Eb = full_mx_exact_exponents<LOG2D>(t_lane, raw_row, a32, tol, near, Eb, i0, p.sqrt_b, lane);
        Eb = min(max(Eb, 0), 254);
        float c;
        if ((LOG2D & 1) == 0) c = __uint_as_float((uint32_t)min(max(254 - Eb - LOG2D / 2, 1), 254) << 23);
        else c = __uint_as_float((uint32_t)min(max(254 - Eb - (LOG2D - 1) / 2, 1), 254) << 23) * 0.70710678118654752f;
        uint32_t byte = (uint32_t)Eb;
        if (!(a32 > 0.0f)) { c = 0.0f; byte = 0u; }
        const float tau = (bref > 0.0f) ? 2.0f * err_rel * bref * c + 2.0e-6f : 0.0f;
        *scale_out = (uint8_t)byte;

        // ---- quantise: both E2M1 code sets, four values at a time
        const f32x2 c2 = pack2(c, c), tp = pack2(tau, tau), tm = pack2(0.0f - tau, 0.0f - tau);
        uint32_t cw[4], tie_any = 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t pw[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int m = 4 * j + 2 * h;
                const f32x2 up0 = fma2(u[m], c2, tp), up1 = fma2(u[m + 1], c2, tp);
                const f32x2 dn0 = fma2(u[m], c2, tm), dn1 = fma2(u[m + 1], c2, tm);
                pw[h] = cvt_e2m1x4_pair(up0.x, up0.y, up1.x, up1.y, dn0.x, dn0.y, dn1.x, dn1.y);
                tie_any |= pw[h] ^ (pw[h] >> 16);
            }
            cw[j] = __byte_perm(pw[0], pw[1], 0x5410);
        }
        *reinterpret_cast<uint4 *>(outp) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        if (__any_sync(0xffffffffu, (tie_any & 0xffffu) != 0u))
            full_mx_fix_ties<LOG2D>(t_lane, raw_row, c, tau, (int)byte, i0, outp, p.sqrt_b, lane);
        __syncwarp();            // the tile is this warp's chunk rows again in the next iteration
        if (++stage == (uint32_t)NST) { stage = 0; parity ^= 1u; }
    }
    if (lane == 0 && !ok) atomicOr(&g_perq_device_error, 1u);
}

}  // namespace perq
