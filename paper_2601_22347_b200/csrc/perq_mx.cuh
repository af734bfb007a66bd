// MXFP4 rotate+quantize kernel with a lean inner loop: unpermuted rows of d % 2048 == 0 channels, Hadamard
// blocks of 16 .. 128, E2M1 codes with one E8M0 scale per 32 rotated values.
//
// Same data path, lane layout, error model and exactness rules as the MXFP4 mode of perq_fast.cuh (whose
// helpers this file uses).  A scale group of 32 never leaves a warp's 1024-element segment, so warps are
// independent; what differs from the group kernel is the loop around a segment.  The kernel is bound by the
// number of instructions it issues, and an iteration's fixed work (the wait for the staged input, the refill
// of the ring, the fence and the bulk store of the packed codes, the loop's bookkeeping) is paid per TWO
// adjacent segments here: a warp's unit is 2048 elements (4 KB in, 1 KB of codes out, one bulk copy each way).
// The rare paths -- a group maximum within the error bound of a power-of-two boundary, an element whose two
// conversions differ -- are functions that are not inlined and that form the rotated values again from the
// staged segment, so that the loop keeps nothing alive for them.
#pragma once
#include "perq_tok.cuh"

namespace perq {

constexpr int MX_SPW = 2;                     // adjacent segments per warp and iteration
constexpr int MX_NSTAGE = 3;                  // ring stages per warp

struct MxSmem {
    static constexpr size_t stages = 0;                                                          // 16 warps x 3 stages x 4 KB
    static constexpr size_t codes = stages + (size_t)FAST_WARPS * MX_NSTAGE * MX_SPW * SEG_BYTES; // 1 KB per warp
    static constexpr size_t full = codes + (size_t)FAST_WARPS * MX_SPW * SEG_CODE_BYTES;          // [16][3] mbarriers
    static constexpr size_t used = full + (size_t)FAST_WARPS * MX_NSTAGE * 8;
    static constexpr size_t total = used + 1024;                                                  // room to align the base
};

// Shared exponent E + 127 (before clamping) of the 32-value group that lane q of a quad owns, from the fp32
// group maximum a32: E = floor(log2(a / sqrt(b))) - 2.  dist is the distance of a32 to the nearest value at
// which that floor changes.
template <int LOG2B>
__device__ __forceinline__ int mx_exponent_fp32(float a32, float &dist)
{
    const uint32_t bits = __float_as_uint(a32);
    const int e8 = (int)(bits >> 23);
    if ((LOG2B & 1) == 0) {
        const float lower = __uint_as_float(bits & 0x7f800000u);
        dist = fminf(a32 - lower, 2.0f * lower - a32);
        return e8 - LOG2B / 2 - 2;
    }
    const uint32_t mant = bits & 0x7fffffu;
    dist = fabsf(a32 - __uint_as_float((bits & 0x7f800000u) | 0x3504f3u));
    return e8 - (LOG2B - 1) / 2 - 3 + (mant >= 0x3504f4u ? 1 : 0);
}

// Pair maxima of a lane's rotated values and the group maximum that lane q of its quad owns (a group of 32 is
// slots 2m, 2m+1 of the four lanes of a quad; lane q owns m = q): a transposed reduction with three shuffles.
__device__ __forceinline__ float mx_group_max(const f32x2 (&v)[8][2], int q, float (&gm)[4])
{
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        float a = max3abs(fabsf(v[2 * m][0].x), v[2 * m][0].y, v[2 * m][1].x);
        a = max3abs(a, v[2 * m][1].y, v[2 * m + 1][0].x);
        a = max3abs(a, v[2 * m + 1][0].y, v[2 * m + 1][1].x);
        gm[m] = fmaxf(a, fabsf(v[2 * m + 1][1].y));
    }
    const bool q1 = (q & 1) != 0, q2 = (q & 2) != 0;
    float k0 = q2 ? gm[2] : gm[0], k1 = q2 ? gm[3] : gm[1];
    const float s0 = q2 ? gm[0] : gm[2], s1 = q2 ? gm[1] : gm[3];
    k0 = fmaxf(k0, __shfl_xor_sync(0xffffffffu, s0, 2));
    k1 = fmaxf(k1, __shfl_xor_sync(0xffffffffu, s1, 2));
    const float keep = q1 ? k1 : k0, send = q1 ? k0 : k1;
    return fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, 1));
}

// Rare: for every group of the segment whose fp32 maximum is within tol of an exponent boundary (near), the
// exact maximum from every element that could attain it, evaluated by the group's quad in fp64; returns the
// lane's exponent (its own group's, if that was one of them).
template <int LOG2B>
__device__ __noinline__ int mx_exact_exponents(uint32_t seg_addr, const uint16_t *seg, float a32, float tol, bool near, int Eb,
                                               double sqrt_b, int lane)
{
    const int q = lane & 3;
    const unsigned qmask = 0xFu << (lane & 28);
    auto over_sqrt_b = [&](double u) -> double {
        return (LOG2B % 2 == 0) ? u * (1.0 / (double)(1 << (LOG2B / 2))) : u / sqrt_b;
    };
    TokLane<LOG2B> L;
    L.init(lane);
    f32x2 v[8][2];
    tok_rotate<LOG2B>(seg_addr, L, v);
    float gm[4];
    (void)mx_group_max(v, q, gm);
    const unsigned near_w = __ballot_sync(0xffffffffu, near);
    const unsigned nearq = (near_w >> (lane & 28)) & 0xFu;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        if ((nearq >> m) & 1u) {
            const int owner = (lane & 28) | m;
            const float a_m = __shfl_sync(qmask, a32, owner), tol_m = __shfl_sync(qmask, tol, owner);
            const float thr = a_m - tol_m;
            const bool has = gm[m] >= thr;
            unsigned cq = __ballot_sync(qmask, has) & qmask;
            double best = 0.0;
            while (cq) {
                const int src = __ffs(cq) - 1;
                cq &= cq - 1;
                uint32_t cm = 0u;
                if (lane == src) {
#pragma unroll
                    for (int mm = 0; mm < 4; ++mm) {
                        if (mm == m) {
                            const float e[8] = {v[2 * mm][0].x, v[2 * mm][0].y, v[2 * mm][1].x, v[2 * mm][1].y,
                                                v[2 * mm + 1][0].x, v[2 * mm + 1][0].y, v[2 * mm + 1][1].x, v[2 * mm + 1][1].y};
#pragma unroll
                            for (int k = 0; k < 8; ++k) cm |= (fabsf(e[k]) >= thr) ? (1u << k) : 0u;
                        }
                    }
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
    return Eb;
}

// The quad's multipliers and windows from the owners' (c, tau), and the two conversions of slot s.
template <int LOG2B>
struct MxQuant {
    f32x2 mulc[8], tau_p[4], tau_m[4];
    __device__ __forceinline__ void init(const TokLane<LOG2B> &L, float c, float tau, int lane)
    {
        constexpr int PM = (1 << (LOG2B - 4)) - 1;
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const float c_m = __shfl_sync(0xffffffffu, c, (lane & 28) | m);
            const float t_m = __shfl_sync(0xffffffffu, tau, (lane & 28) | m);
            tau_p[m] = pack2(t_m, t_m);
            tau_m[m] = pack2(0.0f - t_m, 0.0f - t_m);       // +0 for a zero window: (-0) + (+0) = +0 on both sides
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float mc = L.sgn[(2 * m + h) & 3 & PM] * c_m;
                mulc[2 * m + h] = pack2(mc, mc);
            }
        }
    }
};

// Exact resolution of the elements whose two conversions differ (rare): the rotated values and both code sets
// are formed again from the staged segment; word holds the quad's four scale bytes.
template <int LOG2B>
__device__ __noinline__ void mx_fix_ties(uint32_t seg_addr, const uint16_t *seg, uint8_t *code_gen, float c, float tau, uint32_t word,
                                         double sqrt_b, int lane)
{
    constexpr int B = 1 << LOG2B;
    constexpr int PM = (1 << (LOG2B - 4)) - 1;
    auto over_sqrt_b = [&](double u) -> double {
        return (LOG2B % 2 == 0) ? u * (1.0 / (double)(1 << (LOG2B / 2))) : u / sqrt_b;
    };
    TokLane<LOG2B> L;
    L.init(lane);
    f32x2 v[8][2];
    tok_rotate<LOG2B>(seg_addr, L, v);
    MxQuant<LOG2B> Q;
    Q.init(L, c, tau, lane);
    uint32_t fm = 0u;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const f32x2 up0 = fma2(v[s][0], Q.mulc[s], Q.tau_p[s >> 1]), up1 = fma2(v[s][1], Q.mulc[s], Q.tau_p[s >> 1]);
        const f32x2 dn0 = fma2(v[s][0], Q.mulc[s], Q.tau_m[s >> 1]), dn1 = fma2(v[s][1], Q.mulc[s], Q.tau_m[s >> 1]);
        const uint32_t x0 = cvt_e2m1x2(up0.x, up0.y) ^ cvt_e2m1x2(dn0.x, dn0.y);
        const uint32_t x1 = cvt_e2m1x2(up1.x, up1.y) ^ cvt_e2m1x2(dn1.x, dn1.y);
        fm |= ((x0 & 0x0Fu) ? 1u : 0u) << (4 * s) | ((x0 & 0xF0u) ? 2u : 0u) << (4 * s);
        fm |= ((x1 & 0x0Fu) ? 4u : 0u) << (4 * s) | ((x1 & 0xF0u) ? 8u : 0u) << (4 * s);
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
            const double ue = exact_coord_fast<B>(seg + blk_elem, i, lane);
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

template <int LOG2B>
__global__ void __launch_bounds__(FAST_THREADS, 1) perq_mx_kernel(FastParams p)
{
    static_assert(LOG2B >= 4 && LOG2B <= 7, "blocks inside a segment");
    constexpr int CB = LOG2B - 4;
    constexpr int PM = (1 << CB) - 1;
    constexpr int NST = MX_NSTAGE;
    constexpr uint32_t UNIT_BYTES = (uint32_t)MX_SPW * SEG_BYTES;
    constexpr uint32_t UNIT_ELEMS = (uint32_t)MX_SPW * SEG_ELEMS;
    extern __shared__ __align__(128) unsigned char msmem_raw[];
    unsigned char *msmem = msmem_raw + ((1024u - (smem_u32(msmem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, q = lane & 3;
    const float err_rel = FAST_ERR_K * (float)LOG2B * TWO_M24;

    const uint32_t smem_base = smem_u32(msmem);
    const uint32_t stage_base = smem_base + (uint32_t)MxSmem::stages + (uint32_t)warp * (NST * UNIT_BYTES);
    const uint32_t full_base = smem_base + (uint32_t)MxSmem::full + (uint32_t)warp * (NST * 8);
    const uint32_t code_buf = smem_base + (uint32_t)MxSmem::codes + (uint32_t)warp * (MX_SPW * SEG_CODE_BYTES);

    if (lane < NST) mbar_init(full_base + lane * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    griddep_wait();             // nothing above reads or writes global memory
    griddep_launch();           // the stream's next kernel may be set up on every SM this grid has left (it waits like this one)

    // units of this warp: first, first + stride, ...
    const uint32_t first = blockIdx.x * FAST_WARPS + warp;
    const uint32_t stride = gridDim.x * FAST_WARPS;
    if (first >= p.units_total) return;
    const uint32_t n_units = (p.units_total - first + stride - 1) / stride;
    const uint32_t refill_end = n_units > (uint32_t)NST ? n_units - NST : 0u;

    TokLane<LOG2B> L;
    L.init(lane);
    const size_t unit_step_elems = (size_t)stride * UNIT_ELEMS;
    const uint16_t *xload = p.x + (size_t)first * UNIT_ELEMS;
    uint8_t *outp = p.out_codes + (size_t)first * (MX_SPW * SEG_CODE_BYTES);
    const size_t out_step = (size_t)stride * (MX_SPW * SEG_CODE_BYTES);
    // scale words: 8 per segment (one per lane group: the four bytes of a quad's groups), written by lane q == 0
    uint32_t *scale_out = reinterpret_cast<uint32_t *>(p.out_scales) + (size_t)first * (MX_SPW * 8) + g;
    const size_t scale_step = (size_t)stride * (MX_SPW * 8);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < NST; ++s) {
            if ((uint32_t)s < n_units) {
                mbar_expect_tx(full_base + s * 8, UNIT_BYTES);
                bulk_load(stage_base + s * UNIT_BYTES, xload, UNIT_BYTES, full_base + s * 8);
                xload += unit_step_elems;
            }
        }
    }
    const uint16_t *stage_gen = reinterpret_cast<const uint16_t *>(msmem + MxSmem::stages);
    uint32_t stage = 0, parity = 0;
    bool ok = true;
    for (uint32_t it = 0; it < n_units; ++it, outp += out_step, scale_out += scale_step) {
        const uint32_t bar = full_base + stage * 8;
        if (!mbar_try_once(bar, parity) && !mbar_wait(bar, parity)) { ok = false; break; }
        const uint32_t unit_addr = stage_base + stage * UNIT_BYTES;
        bulk_store_wait_read<0>();           // the store of the previous iteration has read the staging buffer
        __syncwarp();
#pragma unroll
        for (int h = 0; h < MX_SPW; ++h) {
            const uint32_t seg_addr = unit_addr + h * SEG_BYTES;
            f32x2 v[8][2];
            tok_rotate<LOG2B>(seg_addr, L, v);
            float gm[4];
            const float a32 = mx_group_max(v, q, gm);
            // error reference: the largest |u| of the Hadamard block (it may span several groups)
            float bref = a32;
            if (CB >= 2) bref = fmaxf(bref, __shfl_xor_sync(0xffffffffu, bref, 1));
            if (CB >= 3) bref = fmaxf(bref, __shfl_xor_sync(0xffffffffu, bref, 2));
            float dist;
            int Eb = mx_exponent_fp32<LOG2B>(a32, dist);
            const float tol = 2.0f * err_rel * bref + a32 * 2.4e-7f;
            const bool near = (a32 > 0.0f) && (dist <= tol || (__float_as_uint(a32) >> 23) == 0u);
            if (__any_sync(0xffffffffu, near)) {
                const uint16_t *seg = stage_gen + (seg_addr - smem_base - (uint32_t)MxSmem::stages) / 2;
                Eb = mx_exact_exponents<LOG2B>(seg_addr, seg, a32, tol, near, Eb, p.sqrt_b, lane);
            }
            Eb = min(max(Eb, 0), 254);
            // multiplier 2^-E / sqrt(b) and the additive rounding window, in scaled units
            float c;
            if ((LOG2B & 1) == 0) c = __uint_as_float((uint32_t)min(max(254 - Eb - LOG2B / 2, 1), 254) << 23);
            else c = __uint_as_float((uint32_t)min(max(254 - Eb - (LOG2B - 1) / 2, 1), 254) << 23) * 0.70710678118654752f;
            uint32_t byte = (uint32_t)Eb;
            if (!(a32 > 0.0f)) { c = 0.0f; byte = 0u; }
            // (an all-zero block is exact: no window, so that its zeros are not flagged for their sign)
            const float tau = (bref > 0.0f) ? 2.0f * err_rel * bref * c + 2.0e-6f : 0.0f;
            // scale bytes of the quad's four groups: slot pair m is chunk pair m ^ (f >> 1)
            uint32_t word = byte << (8 * (q ^ (((g & 3) & ~PM) >> 1)));
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            if (q == 0) scale_out[h * 8] = word;

            MxQuant<LOG2B> Q;
            Q.init(L, c, tau, lane);
            const uint32_t code_addr0 = code_buf + h * SEG_CODE_BYTES + L.code_lane;
            uint32_t tie_any = 0u;
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const f32x2 up0 = fma2(v[s][0], Q.mulc[s], Q.tau_p[s >> 1]), up1 = fma2(v[s][1], Q.mulc[s], Q.tau_p[s >> 1]);
                const f32x2 dn0 = fma2(v[s][0], Q.mulc[s], Q.tau_m[s >> 1]), dn1 = fma2(v[s][1], Q.mulc[s], Q.tau_m[s >> 1]);
                // both code sets in one word: the low half is stored, the halves are compared
                const uint32_t pw = cvt_e2m1x4_pair(up0.x, up0.y, up1.x, up1.y, dn0.x, dn0.y, dn1.x, dn1.y);
                tie_any |= pw ^ (pw >> 16);
                sts_code<(3 & ~PM)>(code_addr0, s, pw);
            }
            if (__any_sync(0xffffffffu, (tie_any & 0xffffu) != 0u)) {
                const uint16_t *seg = stage_gen + (seg_addr - smem_base - (uint32_t)MxSmem::stages) / 2;
                uint8_t *code_gen = msmem + MxSmem::codes + (code_buf - smem_base - (uint32_t)MxSmem::codes) + h * SEG_CODE_BYTES;
                __syncwarp();
                mx_fix_ties<LOG2B>(seg_addr, seg, code_gen, c, tau, word, p.sqrt_b, lane);
            }
        }
        // ---- packed codes of both segments: shared staging -> global; the stage is free again
        fence_async_smem();
        __syncwarp();
        bulk_store_if(lane == 0, outp, code_buf, MX_SPW * SEG_CODE_BYTES);
        {
            const bool go = (lane == 0) && (it < refill_end);           // unit it + NST exists
            bulk_load_if(go, unit_addr, xload, UNIT_BYTES, bar);
            if (go) xload += unit_step_elems;
        }
        if (++stage == (uint32_t)NST) { stage = 0; parity ^= 1u; }
    }
    if (lane == 0 && !ok) atomicOr(&g_perq_device_error, 1u);
    bulk_store_wait_read<0>();
}

}  // namespace perq
