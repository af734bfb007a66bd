// Per-token rotate+quantize kernel with a lean inner loop: unpermuted rows of d = 2048, 4096 or 8192
// channels, Hadamard blocks of 16 .. 128, symmetric INT4 or E2M1 codes with one fp32 scale per token.
//
// Same data path, lane layout, error model and exactness rules as perq_fast.cuh (whose helpers it uses).
// What differs is the loop around a segment: this path is bound by the number of warp instructions it issues
// (measured: 0.1 to 0.2 us of a 16384 x 4096 call per instruction and 1024-element segment), and a good half
// of the group kernel's instructions were not the rotation, the maxima or the quantiser:
//
//   * A warp owns two adjacent 1024-element segments of a row, and a row is shared by W = d / 2048 warps.
//     What an iteration costs once -- the wait for the staged row, the exchange of maxima around the row's
//     named barrier, the refill of the ring, the fence and the bulk store of the packed codes, the loop's
//     own bookkeeping: about a hundred instructions -- is paid per two segments.  The first segment's rotated
//     values are not kept while the second one's maximum is formed: it is rotated again (28 instructions)
//     after the second one is quantised.
//   * The warps of a row share nothing but their fp32 maxima (one 4-byte word each, exchanged around the
//     row's named barrier).  The warp that holds the row maximum pins it to one lane and one pair of slots
//     (8 outputs) from the four pair maxima it has anyway, and appends a record; the exact scale is derived
//     later, one record per lane, from the bf16 inputs in global memory.
//   * Whoever needs the exact row maximum at once -- a row whose maximum is not pinned down that way, a warp
//     with an element whose two-sided rounding test failed -- derives it itself from the staged row, in a
//     function that is not inlined and that forms the rotated values again.  Nothing is published, no flag is
//     waited for, and the loop keeps nothing alive for the rare paths.
//   * Addresses advance by increments; the asynchronous copies are predicated inside their PTX blocks (no
//     branch around them); waits take the bounded slow path only when the first poll fails.
#pragma once
#include "perq_fast.cuh"

namespace perq {

constexpr int TOK_SPW = 2;                    // adjacent segments of a row per warp
constexpr int TOK_NSTAGE = 3;                 // ring stages (rows) per group of warps

// Shared memory, relative to a 1024-byte aligned base: 16 warps x 3 stages x 2 segments of 2 KB, one 1 KB
// code staging buffer per warp, the ring's mbarriers, the warp maxima, the deferred scale records.
struct TokSmem {
    static constexpr size_t stages = 0;
    static constexpr size_t codes = stages + (size_t)FAST_WARPS * TOK_NSTAGE * TOK_SPW * SEG_BYTES;
    static constexpr size_t full = codes + (size_t)FAST_WARPS * TOK_SPW * SEG_CODE_BYTES;
    static constexpr size_t xch = full + (size_t)FAST_WARPS * TOK_NSTAGE * 8;            // [2][16] fp32 warp maxima (8 bytes apart)
    static constexpr size_t wreq = xch + (size_t)2 * FAST_WARPS * 8;                     // [16][16] u64 deferred scale records
    static constexpr size_t used = wreq + (size_t)FAST_WARPS * 16 * 8;
    static constexpr size_t total = used + 1024;                                         // room to align the base
};
constexpr uint32_t TOK_MAX_RECORDS = 16;

// Per-lane constants of the data layout (see perq_fast.cuh): Hadamard operand of the tensor-core stage,
// ldmatrix source offset, position of the lane's code piece, relabelling signs.
template <int LOG2B>
struct TokLane {
    uint32_t hb[2][2];
    uint32_t lm0;
    uint32_t code_lane;
    float sgn[4];
    __device__ __forceinline__ void init(int lane)
    {
        constexpr int PM = (1 << (LOG2B - 4)) - 1;
        const int g = lane >> 2, q = lane & 3;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const int col = 4 * (g >> 1) + (g & 1) + 2 * m;
            hb[m][0] = hadamard_bf16(2 * q, col) | (hadamard_bf16(2 * q + 1, col) << 16);
            hb[m][1] = hadamard_bf16(2 * q + 8, col) | (hadamard_bf16(2 * q + 9, col) << 16);
        }
        const int r8 = lane & 7, mi = lane >> 3;
        const int f = r8 & 3, fh = (r8 >> 2) & 1;
        lm0 = (uint32_t)((r8 * 8 + ((mi & 1) ^ f)) * 32 + (((mi >> 1) ^ fh) * 16));
        const int f_g = g & 3;
        code_lane = (uint32_t)((g * 8 + (f_g & ~PM)) * 8 + 2 * q);
        const float half_sign = ((g & 4) && q >= 2) ? -1.0f : 1.0f;
#pragma unroll
        for (int k = 0; k < 4; ++k) sgn[k] = (__popc(k & f_g & PM) & 1) ? -half_sign : half_sign;
    }
};

// The rotated values of the segment at shared address seg_addr: v[s][h] = outputs (2h, 2h+1) of this
// lane's four of slot s, up to the relabelling signs.
template <int LOG2B>
__device__ __forceinline__ void tok_rotate(uint32_t seg_addr, const TokLane<LOG2B> &L, f32x2 (&v)[8][2])
{
    constexpr int CB = LOG2B - 4;
    const uint32_t a0 = seg_addr + L.lm0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        uint32_t a[4];
        if (t & 2) ldmatrix_x4_at<128>(a, a0 ^ (uint32_t)((t & 1) << 6));
        else ldmatrix_x4_at<0>(a, a0 ^ (uint32_t)((t & 1) << 6));
        float c0[4], c1[4];
        mma_bf16(c0, a, L.hb[0][0], L.hb[0][1]);
        mma_bf16(c1, a, L.hb[1][0], L.hb[1][1]);
        v[2 * t][0] = pack2(c0[0], c0[1]);
        v[2 * t][1] = pack2(c1[0], c1[1]);
        v[2 * t + 1][0] = pack2(c0[2], c0[3]);
        v[2 * t + 1][1] = pack2(c1[2], c1[3]);
    }
#pragma unroll
    for (int t = 0; t < CB; ++t) {
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            if ((s & (1 << t)) == 0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const f32x2 a = v[s][h], c = v[s | (1 << t)][h];
                    v[s][h] = add2(a, c);
                    v[s | (1 << t)][h] = sub2(a, c);
                }
            }
        }
    }
}

__device__ __forceinline__ bool mbar_try_once(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0u;
}

// One lane's asynchronous copies, predicated inside the PTX block so that no branch surrounds them.
__device__ __forceinline__ void bulk_load_if(bool pred, uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("{ .reg .pred p; setp.ne.u32 p, %4, 0;\n"
                 "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], %2;\n"
                 "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3]; }"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "r"((uint32_t)pred) : "memory");
}
__device__ __forceinline__ void bulk_store_if(bool pred, void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("{ .reg .pred p; setp.ne.u32 p, %3, 0;\n"
                 "@p cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n"
                 "@p cp.async.bulk.commit_group; }" ::"l"(dst), "r"(src), "r"(bytes), "r"((uint32_t)pred) : "memory");
}

// Largest magnitude of the eight outputs i0 .. i0+3 and i0+16 .. i0+19 (the lane's outputs of a pair of
// chunks) around position pos of a row in global memory; pos is a multiple of 4 with bit 4 clear.  One thread,
// fp64: the sums are exact.  For blocks of 32 and more both slots lie in one block and share the partial
// sums (terms with k & 3 == e, split by bit 4 of k); blocks of 16 are two blocks.
template <int LOG2B>
__device__ __forceinline__ double exact_pair_max_global(const uint16_t *row, uint32_t pos)
{
    constexpr int B = 1 << LOG2B;
    if (LOG2B == 4) {
        double best = 0.0;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const uint32_t ps = pos + 16u * half;
            const uint4 *src = reinterpret_cast<const uint4 *>(row + (ps & ~15u));
            const uint32_t i0 = ps & 15u;
            double S[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const uint4 w4 = __ldg(src + c);
                const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
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
            best = fmax(best, fmax(fmax(fabs(a0 + a2), fabs(a1 + a3)), fmax(fabs(a0 - a2), fabs(a1 - a3))));
        }
        return best;
    }
    const uint32_t blk = (pos >> LOG2B) << LOG2B;
    const uint32_t i0 = pos - blk;                       // bit 4 clear
    const uint4 *src = reinterpret_cast<const uint4 *>(row + blk);
    double Sl[4] = {0.0, 0.0, 0.0, 0.0}, Sh[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll 2
    for (int c2 = 0; c2 < B / 16; ++c2) {               // sixteen inputs at a time: bit 4 of k is bit 0 of c2
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            const int c = 2 * c2 + cc;
            const uint4 w4 = __ldg(src + c);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const bool neg = __popc(i0 & (uint32_t)(8 * c + 4 * h)) & 1;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t word = w[2 * h + (e >> 1)];
                    const double val = (double)__uint_as_float((e & 1) ? (word & 0xffff0000u) : (word << 16));
                    const double sv = neg ? -val : val;
                    if (c2 & 1) Sh[e] += sv; else Sl[e] += sv;
                }
            }
        }
    }
    double best = 0.0;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        double S[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) S[e] = half ? Sl[e] - Sh[e] : Sl[e] + Sh[e];
        const double a0 = S[0] + S[1], a1 = S[0] - S[1], a2 = S[2] + S[3], a3 = S[2] - S[3];
        best = fmax(best, fmax(fmax(fabs(a0 + a2), fabs(a1 + a3)), fmax(fabs(a0 - a2), fabs(a1 - a3))));
    }
    return best;
}

// Deferred per-token scales: record = row << 32 | pair position in the row; one record per lane.
template <int LOG2B>
__device__ __noinline__ void tok_serve_records(const uint16_t *x, float *out_scales, int d, double inv_7_sqrt_b,
                                               const unsigned long long *req, uint32_t n, int lane)
{
    __syncwarp();
    if ((uint32_t)lane < n) {
        const unsigned long long r = req[lane];
        const uint32_t row = (uint32_t)(r >> 32), pos = (uint32_t)r;
        const double a = exact_pair_max_global<LOG2B>(x + (size_t)row * d, pos);
        out_scales[row] = (a == 0.0) ? 0.0f : (float)(a * inv_7_sqrt_b);
    }
    __syncwarp();
}

// The exact largest magnitude of a staged row (bit pattern of a non-negative double, the same in every
// lane), by one warp: every segment of a warp whose fp32 maximum is within the error bound of the row's is
// rotated again and its candidate slots are evaluated in fp64 from the bf16 inputs.  xch holds the fp32
// maxima of the row's W warps, 8 bytes apart (W = 1: not read); a warp owns TOK_SPW adjacent segments.
// Rare: rows whose maximum is not pinned to one pair of slots, and warps that need the exact maximum for
// a fix-up.
template <int LOG2B, int LOG2W>
__device__ __noinline__ unsigned long long tok_row_exact_max(uint32_t row_addr, const uint16_t *raw_row, const uint32_t *xch,
                                                             float thr_row, int lane)
{
    constexpr int W = 1 << LOG2W;
    TokLane<LOG2B> L;
    L.init(lane);
    unsigned long long best = 0ull;
#pragma unroll 1
    for (int sgm = 0; sgm < W * TOK_SPW; ++sgm) {
        if (W > 1 && !(__uint_as_float(xch[2 * (sgm / TOK_SPW)]) >= thr_row)) continue;
        f32x2 v[8][2];
        tok_rotate<LOG2B>(row_addr + (uint32_t)sgm * SEG_BYTES, L, v);
        float ms[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) ms[s] = fmaxf(max3abs(fabsf(v[s][0].x), v[s][0].y, v[s][1].x), fabsf(v[s][1].y));
        const unsigned long long wb = exact_max_of_candidates<LOG2B, 0>(raw_row + (size_t)sgm * SEG_ELEMS, 0, ms, thr_row, lane);
        best = wb > best ? wb : best;
    }
    return best;
}

// Exact resolution of the elements whose two-sided rounding test failed (rare).  The rotated values and
// the two code sets are formed again from the staged segment; the exact row maximum, unless this warp has it
// already (known), is derived from the staged row.
template <int LOG2B, int MODE, int LOG2W>
__device__ __noinline__ void tok_fix_ties(uint32_t seg_addr, const uint16_t *seg, uint32_t row_addr, const uint16_t *raw_row,
                                          const uint32_t *xch, uint8_t *code_gen, float inv, float a32, float thr_row,
                                          double sqrt_b, bool known, unsigned long long a_bits, int lane)
{
    constexpr int B = 1 << LOG2B;
    constexpr int PM = (1 << (LOG2B - 4)) - 1;
    constexpr float MAGIC = 12582920.0f;
    const float err_rel = FAST_ERR_K * (float)LOG2B * TWO_M24;
    auto over_sqrt_b = [&](double u) -> double {
        return (LOG2B % 2 == 0) ? u * (1.0 / (double)(1 << (LOG2B / 2))) : u / sqrt_b;
    };
    TokLane<LOG2B> L;
    L.init(lane);
    f32x2 v[8][2];
    tok_rotate<LOG2B>(seg_addr, L, v);
    const float delta = 16.0f * err_rel + 5.0e-7f;
    const float tau = (a32 > 0.0f) ? 8.0f * err_rel + 4.0e-6f : 0.0f;
    const f32x2 magic2 = pack2(MAGIC, MAGIC);
    const f32x2 tau_p2 = pack2(tau, tau), tau_m2 = pack2(0.0f - tau, 0.0f - tau);     // (+0 for a zero row)
    uint32_t fm = 0u, zm = 0u;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const int c = s & 3 & PM;
        if (MODE == MODE_FP4) {
            const float mc = L.sgn[c] * inv;
            const f32x2 mc2 = pack2(mc, mc);
            const f32x2 up0 = fma2(v[s][0], mc2, tau_p2), up1 = fma2(v[s][1], mc2, tau_p2);
            const f32x2 dn0 = fma2(v[s][0], mc2, tau_m2), dn1 = fma2(v[s][1], mc2, tau_m2);
            const uint32_t x = cvt_e2m1x4(up0.x, up0.y, up1.x, up1.y) ^ cvt_e2m1x4(dn0.x, dn0.y, dn1.x, dn1.y);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t xn = (x >> (4 * e)) & 0xFu;
                fm |= xn ? (1u << (4 * s + e)) : 0u;
                zm |= (xn == 8u) ? (1u << (4 * s + e)) : 0u;      // the codes differ in the sign alone
            }
        } else {
            const float mp = L.sgn[c] * inv * (1.0f + delta), mm = L.sgn[c] * inv * (1.0f - delta);
            const f32x2 mp2 = pack2(mp, mp), mm2 = pack2(mm, mm);
            const f32x2 tp0 = fma2(v[s][0], mp2, magic2), tp1 = fma2(v[s][1], mp2, magic2);
            const f32x2 tm0 = fma2(v[s][0], mm2, magic2), tm1 = fma2(v[s][1], mm2, magic2);
            const float t[4] = {tp0.x, tp0.y, tp1.x, tp1.y}, u[4] = {tm0.x, tm0.y, tm1.x, tm1.y};
#pragma unroll
            for (int e = 0; e < 4; ++e) fm |= (t[e] != u[e]) ? (1u << (4 * s + e)) : 0u;
        }
    }
    // The exact row maximum a.  E2M1 codes need it unless only signs are in doubt.  INT4 codes mostly do not:
    // the fp32 maximum a32 brackets it, a32 (1 - a_unc) <= a <= a32 (1 + a_unc) (the largest fp32 value and the
    // largest exact value are both within the error bound of each other's element), which decides every element
    // that is not within that bracket of its tie -- about fifteen in sixteen of the elements that get here,
    // whose window is sixteen times wider.  It is derived from the staged row only when an element asks for it.
    const float a_unc = 1.0625f * err_rel + 2.4e-7f;
    if (MODE == MODE_FP4) {
        // The zeros of an all-zero block (padded channels) are exact, and the staged code +0 is theirs: drop
        // their flags (the window of the loop's test is the same for every block of the row).  A block is 2^CB
        // slots of the four lanes of a quad.
        constexpr int CB = LOG2B - 4;
        float bm[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) bm[s] = fmaxf(max3abs(fabsf(v[s][0].x), v[s][0].y, v[s][1].x), fabsf(v[s][1].y));
#pragma unroll
        for (int s = 0; s < 8; s += (1 << CB)) {
            float m = bm[s];
#pragma unroll
            for (int k = 1; k < (1 << CB); ++k) m = fmaxf(m, bm[s + k]);
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            if (m == 0.0f) {
#pragma unroll
                for (int k = 0; k < (1 << CB); ++k) fm &= ~(0xFu << (4 * (s + k)));
            }
        }
        if (!__any_sync(0xffffffffu, fm != 0u)) return;
    }
    if (MODE == MODE_FP4 && !known && __any_sync(0xffffffffu, (fm & ~zm) != 0u)) {
        a_bits = tok_row_exact_max<LOG2B, LOG2W>(row_addr, raw_row, xch, thr_row, lane);
        known = true;
    }
    __syncwarp();
    double s_row = 0.0;
    bool have_s = false;
    unsigned tl = __ballot_sync(0xffffffffu, fm != 0u);
    while (tl) {
        const int src = __ffs(tl) - 1;
        tl &= tl - 1;
        uint32_t fs = __shfl_sync(0xffffffffu, fm, src);
        const uint32_t zs = __shfl_sync(0xffffffffu, zm, src);
        while (fs) {
            const int e = __ffs(fs) - 1;
            fs &= fs - 1;
            int blk_elem, i, elem;
            locate<LOG2B>(src >> 2, src & 3, e, blk_elem, i, elem);
            // (lane 0's sum for everybody: the lanes add in different orders, and the branches below must not differ)
            const double ue = __shfl_sync(0xffffffffu, exact_coord_fast<B>(seg + blk_elem, i, lane), 0);
            uint32_t code = 0u;
            if (MODE == MODE_FP4) {
                if ((zs >> e) & 1u) {
                    code = signbit(ue) ? 8u : 0u;          // magnitude zero either way: the sign of y = u / sqrt(b)
                } else {
                    const double a_src = __longlong_as_double((long long)a_bits);
                    if (!have_s) { s_row = over_sqrt_b(a_src) / 7.0; have_s = true; }
                    const double y = over_sqrt_b(ue);
                    code = e2m1_code_exact((s_row != 0.0) ? y / s_row : 0.0, signbit(y));
                }
            } else if (a32 > 0.0f) {
                // The staged code kp comes from the multiplier nudged away from zero, the other candidate is one
                // step towards zero, the tie between them at |y / s| = |kp| - 1/2.  y / s = 7 u / a: the side is the
                // sign of 14 |u| - (2 |kp| - 1) a, two fp64 products whose rounding errors are far below the margins
                // asked for here.  Only an exact or all but exact tie takes the definition's own sequence of
                // operations (fp64 divisions), which lands on exact halves where the definition does.
                // (read by one lane and handed round: every lane takes the same branches below, and none reads the
                // byte after lane 0 has rewritten it)
                const uint32_t nib = __shfl_sync(0xffffffffu, (uint32_t)(code_gen[elem >> 1] >> ((elem & 1) * 4)) & 0xFu, 0);
                const int kp = (int)(nib ^ 8u) - 8;
                const int mag = kp < 0 ? -kp : kp;
                const double lhs = 14.0 * fabs(ue), wgt = (double)(2 * mag - 1);
                const uint32_t towards_zero = (uint32_t)(kp < 0 ? kp + 1 : kp - 1) & 0xFu;
                bool decided = false;
                if (!known && mag >= 1) {
                    const double d32 = lhs - wgt * (double)a32;
                    if (fabs(d32) > wgt * (double)a32 * (double)a_unc) {
                        code = d32 > 0.0 ? ((uint32_t)kp & 0xFu) : towards_zero;
                        decided = true;
                    }
                }
                if (!decided) {                            // (warp-uniform: every lane holds the same operands)
                    if (!known) {
                        a_bits = tok_row_exact_max<LOG2B, LOG2W>(row_addr, raw_row, xch, thr_row, lane);
                        known = true;
                    }
                    const double a_src = __longlong_as_double((long long)a_bits);
                    const double diff = lhs - wgt * a_src;
                    if (mag >= 1 && fabs(diff) > a_src * 1.0e-12) {
                        code = diff > 0.0 ? ((uint32_t)kp & 0xFu) : towards_zero;
                    } else if (a_src != 0.0) {
                        if (!have_s) { s_row = over_sqrt_b(a_src) / 7.0; have_s = true; }
                        double qd = rint(over_sqrt_b(ue) / s_row);
                        qd = fmin(fmax(qd, -8.0), 7.0);
                        code = (uint32_t)((int)qd) & 0xFu;
                    }
                }
            }
            if (lane == 0) {
                uint8_t *bp = code_gen + (elem >> 1);
                *bp = (elem & 1) ? (uint8_t)((*bp & 0x0F) | (code << 4)) : (uint8_t)((*bp & 0xF0) | code);
            }
            __syncwarp();
        }
    }
}

template <int LOG2B, int MODE, int LOG2W>
__global__ void __launch_bounds__(FAST_THREADS, 1) perq_tok_kernel(FastParams p)
{
    static_assert(MODE == MODE_TOKEN || MODE == MODE_FP4, "one scale per token");
    static_assert(LOG2B >= 4 && LOG2B <= 7 && LOG2W >= 0 && LOG2W <= 2, "blocks inside a segment, rows of 2, 4 or 8 segments");
    constexpr int W = 1 << LOG2W;                 // warps per row
    constexpr int GROUPS = FAST_WARPS / W;
    constexpr int PM = (1 << (LOG2B - 4)) - 1;
    constexpr int NCLS = (PM & 3) + 1;
    constexpr int NST = TOK_NSTAGE;
    constexpr uint32_t UNIT_BYTES = (uint32_t)(W * TOK_SPW) * SEG_BYTES;
    constexpr uint32_t UNIT_ELEMS = (uint32_t)(W * TOK_SPW) * SEG_ELEMS;
    constexpr float MAGIC = 12582920.0f;          // 1.5 * 2^23 + 8: low nibble of the sum = code + 8
    extern __shared__ __align__(128) unsigned char tsmem_raw[];
    unsigned char *tsmem = tsmem_raw + ((1024u - (smem_u32(tsmem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = warp >> LOG2W;
    // position in the row, rotated by the group index (the same position of every row tends to do the per-row
    // extra work; warps go to the four schedulers by warp index)
    const int w_in_g = (warp + group) & (W - 1);
    const float err_rel = FAST_ERR_K * (float)LOG2B * TWO_M24;
    const float thr_factor = 1.0f - 2.0f * err_rel - 2.4e-7f;
    const float delta = 16.0f * err_rel + 5.0e-7f;

    const uint32_t smem_base = smem_u32(tsmem);
    const uint32_t stage_base = smem_base + (uint32_t)TokSmem::stages + (uint32_t)group * (NST * UNIT_BYTES);
    const uint32_t seg_base = stage_base + (uint32_t)w_in_g * (TOK_SPW * SEG_BYTES);
    const uint32_t full_base = smem_base + (uint32_t)TokSmem::full + (uint32_t)group * (NST * 8);
    const uint32_t code_buf = smem_base + (uint32_t)TokSmem::codes + (uint32_t)warp * (TOK_SPW * SEG_CODE_BYTES);
    const uint32_t xch_group = smem_base + (uint32_t)TokSmem::xch + (uint32_t)(group * W) * 8;
    unsigned long long *wreq = reinterpret_cast<unsigned long long *>(tsmem + TokSmem::wreq) + warp * TOK_MAX_RECORDS;

    if (tid < FAST_WARPS * NST) mbar_init(smem_base + (uint32_t)TokSmem::full + tid * 8, 1);
    if (tid == 0) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    griddep_wait();             // nothing above reads or writes global memory
    griddep_launch();           // the stream's next kernel may be set up on every SM this grid has left (it waits like this one)

    const uint32_t first = blockIdx.x * GROUPS + group;
    const uint32_t stride = gridDim.x * GROUPS;
    if (first >= p.units_total) return;          // whole groups leave together
    const uint32_t n_units = (p.units_total - first + stride - 1) / stride;
    const uint32_t refill_end = n_units > (uint32_t)NST ? n_units - NST : 0u;     // iterations 1 .. refill_end load a row
    const bool leader = (w_in_g == 0) && (lane == 0);

    TokLane<LOG2B> L;
    L.init(lane);
    // quantisation multipliers per sign class, up to the row's factor 7 / |y|max (a sign change is exact, so
    // inv * (sgn * (1 +- delta)) are the same floats as (sgn * inv) * (1 +- delta))
    float cp[NCLS], cm[NCLS];
#pragma unroll
    for (int c = 0; c < NCLS; ++c) { cp[c] = L.sgn[c] * (1.0f + delta); cm[c] = L.sgn[c] * (1.0f - delta); }

    // running addresses
    const size_t unit_step_elems = (size_t)stride * UNIT_ELEMS;
    const uint16_t *xload = p.x + (size_t)first * UNIT_ELEMS;                  // leader: source of the next row to load
    uint8_t *outp = p.out_codes + ((size_t)first * (W * TOK_SPW) + (size_t)w_in_g * TOK_SPW) * SEG_CODE_BYTES;
    const size_t out_step = (size_t)stride * (W * TOK_SPW) * SEG_CODE_BYTES;
    float *scales = reinterpret_cast<float *>(p.out_scales);
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
    uint32_t xch_it = xch_group;                 // this iteration's exchange words: two sets alternate
    uint32_t stage = 0, parity = 0;              // ring position of this iteration

    // magnitude maxima of the four slot pairs of a segment's rotated values
    auto pair_maxima = [&](const f32x2 (&v)[8][2], float (&gm)[4]) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            float a = max3abs(fabsf(v[2 * m][0].x), v[2 * m][0].y, v[2 * m][1].x);
            a = max3abs(a, v[2 * m][1].y, v[2 * m + 1][0].x);
            a = max3abs(a, v[2 * m + 1][0].y, v[2 * m + 1][1].x);
            gm[m] = fmaxf(a, fabsf(v[2 * m + 1][1].y));
        }
    };
    // Quantise a segment's rotated values into the staging buffer at code_addr0 (+ this lane's offset):
    // packed fp32 multiply-add against the magic constant, with the multiplier nudged up and down by the
    // error bound (E2M1: the scaled value plus and minus an additive window, converted twice).  Returns the
    // OR of the differences between the two code sets.
    auto quantise = [&](const f32x2 (&v)[8][2], float inv, uint32_t code_addr0) -> uint32_t {
        uint32_t tie_any = 0u;
        if (MODE == MODE_FP4) {
            const float tau = (inv > 0.0f) ? 8.0f * err_rel + 4.0e-6f : 0.0f;
            const f32x2 tau_p2 = pack2(tau, tau), tau_m2 = pack2(0.0f - tau, 0.0f - tau);     // (+0 for a zero row)
            f32x2 mul_c[NCLS];
#pragma unroll
            for (int c = 0; c < NCLS; ++c) mul_c[c] = pack2(L.sgn[c] * inv, L.sgn[c] * inv);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int c = s & 3 & PM;
                const f32x2 up0 = fma2(v[s][0], mul_c[c], tau_p2), up1 = fma2(v[s][1], mul_c[c], tau_p2);
                const f32x2 dn0 = fma2(v[s][0], mul_c[c], tau_m2), dn1 = fma2(v[s][1], mul_c[c], tau_m2);
                const uint32_t pu = cvt_e2m1x4(up0.x, up0.y, up1.x, up1.y);
                const uint32_t pd = cvt_e2m1x4(dn0.x, dn0.y, dn1.x, dn1.y);
                tie_any |= pu ^ pd;
                sts_code<(3 & ~PM)>(code_addr0, s, pu);
            }
        } else {
            f32x2 mul_p[NCLS], mul_m[NCLS];
#pragma unroll
            for (int c = 0; c < NCLS; ++c) {
                const float mp = inv * cp[c], mm = inv * cm[c];
                mul_p[c] = pack2(mp, mp);
                mul_m[c] = pack2(mm, mm);
            }
            const f32x2 magic2 = pack2(MAGIC, MAGIC);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int c = s & 3 & PM;
                const f32x2 tp0 = fma2(v[s][0], mul_p[c], magic2), tp1 = fma2(v[s][1], mul_p[c], magic2);
                const f32x2 tm0 = fma2(v[s][0], mul_m[c], magic2), tm1 = fma2(v[s][1], mul_m[c], magic2);
                const uint32_t pp = ((__float_as_uint(tp1.y) * 16u + __float_as_uint(tp1.x)) * 16u + __float_as_uint(tp0.y)) * 16u
                                    + __float_as_uint(tp0.x);
                const uint32_t pm = ((__float_as_uint(tm1.y) * 16u + __float_as_uint(tm1.x)) * 16u + __float_as_uint(tm0.y)) * 16u
                                    + __float_as_uint(tm0.x);
                tie_any |= pp ^ pm;          // low 16 bits: the four codes (offset by 8) under either multiplier
                sts_code<(3 & ~PM)>(code_addr0, s, pp ^ 0x8888u);
            }
        }
        return tie_any & 0xffffu;
    };

    uint32_t nreq = 0;                           // records waiting in wreq (the same in every lane)
    uint32_t unit = first;
    bool ok = true;
    for (uint32_t it = 0; it < n_units; ++it, unit += stride, outp += out_step, xch_it ^= FAST_WARPS * 8) {
        const uint32_t bar = full_base + stage * 8;
        if (!mbar_try_once(bar, parity) && !mbar_wait(bar, parity)) { ok = false; break; }
        const uint32_t row_addr = stage_base + stage * UNIT_BYTES;
        const uint32_t seg_addr = seg_base + stage * UNIT_BYTES;          // this warp's first segment; the second follows

        // ---- first segment: pair maxima only; second segment: its rotated values stay
        f32x2 v[8][2];
        float gm[2][4];
        tok_rotate<LOG2B>(seg_addr, L, v);
        pair_maxima(v, gm[0]);
        tok_rotate<LOG2B>(seg_addr + SEG_BYTES, L, v);
        pair_maxima(v, gm[1]);
        // (a tournament, whose intermediate winners the candidate warp uses again below)
        const float q0 = fmaxf(gm[0][0], gm[0][1]), q1 = fmaxf(gm[0][2], gm[0][3]);
        const float q2 = fmaxf(gm[1][0], gm[1][1]), q3 = fmaxf(gm[1][2], gm[1][3]);
        const float s0 = fmaxf(q0, q1), s1 = fmaxf(q2, q3);
        const float lane_max = fmaxf(s0, s1);
        const float aw = warp_max_f32(lane_max);
        float a32 = aw;
        if (W > 1) {
            if (lane == 0) asm volatile("st.shared.b32 [%0], %1;" ::"r"(xch_it + (uint32_t)w_in_g * 8), "r"(__float_as_uint(aw)) : "memory");
            named_barrier(1 + group, W * 32);
            uint32_t am_bits;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(am_bits) : "r"(xch_it + (uint32_t)(lane & (W - 1)) * 8) : "memory");
            a32 = warp_max_f32(__uint_as_float(am_bits));          // (every lane reads one of the row's W words)
        }
        // every warp of the group is past the stage of the previous iteration: lane 0 of the first warp refills it
        if (w_in_g == 0) {
            const uint32_t ps = stage == 0 ? (uint32_t)(NST - 1) : stage - 1u;
            const bool go = (lane == 0) && (it - 1u < refill_end);     // it >= 1 and row it + NST - 1 exists (it - 1 wraps for it == 0)
            bulk_load_if(go, stage_base + ps * UNIT_BYTES, xload, UNIT_BYTES, full_base + ps * 8);
            if (go) xload += unit_step_elems;
        }
        const float thr_row = a32 * thr_factor;

        // ---- the warp that holds the row maximum: pin it to one lane and one pair of slots, record it
        bool known = !(a32 > 0.0f);              // this warp holds the exact row maximum in a_bits
        unsigned long long a_bits = 0ull;
        if (aw >= thr_row) {
            if (a32 > 0.0f) {
                bool pinned = false;
                if (W == 1 || aw == a32) {       // (ties between warps and near ties take the general path below)
                    const unsigned cl = __ballot_sync(0xffffffffu, lane_max >= thr_row);
                    // the largest of the tournament's seven losers is the lane's second largest pair maximum
                    const float r01 = fmaxf(fminf(gm[0][0], gm[0][1]), fminf(gm[0][2], gm[0][3]));
                    const float r23 = fmaxf(fminf(gm[1][0], gm[1][1]), fminf(gm[1][2], gm[1][3]));
                    const float second = fmaxf(fmaxf(r01, r23), fmaxf(fmaxf(fminf(q0, q1), fminf(q2, q3)), fminf(s0, s1)));
                    // index 4h + m of the one pair maximum that reaches the bound (meaningless if there are several)
                    const uint32_t idx = (s1 >= thr_row ? 4u : 0u) | ((q1 >= thr_row || q3 >= thr_row) ? 2u : 0u) |
                                         ((gm[0][1] >= thr_row || gm[0][3] >= thr_row || gm[1][1] >= thr_row || gm[1][3] >= thr_row) ? 1u : 0u);
                    const int src = __ffs(cl) - 1;
                    const uint32_t packed = __shfl_sync(0xffffffffu, idx | (second < thr_row ? 16u : 0u), src & 31);
                    bool alone = (cl & (cl - 1)) == 0u && (packed >> 4) == 1u;
                    if (W > 1) {                 // no other warp of the row within the bound
                        uint32_t ob;
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(ob) : "r"(xch_it + (uint32_t)(lane & (W - 1)) * 8) : "memory");
                        alone = alone && __popc(__ballot_sync(0xffffffffu, lane < W && __uint_as_float(ob) >= thr_row)) == 1;
                    }
                    if (alone) {
                        // slots 2m, 2m+1 of lane group sg are the chunks 8 sg + ((2m, 2m+1) ^ relabelling): one aligned pair
                        const uint32_t sg = (uint32_t)src >> 2, m = packed & 3u, h = (packed >> 2) & 1u;
                        const uint32_t chunk = sg * 8 + (((2 * m) ^ (sg & 3u & ~(uint32_t)PM)) & ~1u);
                        const uint32_t pos = (uint32_t)(w_in_g * TOK_SPW + h) * SEG_ELEMS + chunk * 16 + 4 * ((uint32_t)src & 3u);
                        if (lane == 0) wreq[nreq] = ((unsigned long long)unit << 32) | pos;
                        if (++nreq == TOK_MAX_RECORDS) {
                            tok_serve_records<LOG2B>(p.x, scales, p.d, p.inv_7_sqrt_b, wreq, nreq, lane);
                            nreq = 0;
                        }
                        pinned = true;
                    }
                }
                if (!pinned) {
                    // several candidates: the first warp of the row that is within the bound derives the exact
                    // maximum of the whole row and stores the scale
                    bool mine = true;
                    if (W > 1) {
                        uint32_t ob;
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(ob) : "r"(xch_it + (uint32_t)(lane & (W - 1)) * 8) : "memory");
                        const unsigned cw = __ballot_sync(0xffffffffu, lane < W && __uint_as_float(ob) >= thr_row);
                        mine = (__ffs(cw) - 1) == w_in_g;
                    }
                    if (mine) {
                        const uint16_t *raw_row = reinterpret_cast<const uint16_t *>(tsmem + TokSmem::stages) + (row_addr - smem_base - (uint32_t)TokSmem::stages) / 2;
                        a_bits = tok_row_exact_max<LOG2B, LOG2W>(row_addr, raw_row, reinterpret_cast<const uint32_t *>(tsmem + TokSmem::xch) + (xch_it - smem_base - (uint32_t)TokSmem::xch) / 4,
                                                                 thr_row, lane);
                        known = true;
                        if (lane == 0) scales[unit] = (a_bits == 0ull) ? 0.0f : (float)(__longlong_as_double((long long)a_bits) * p.inv_7_sqrt_b);
                    }
                }
            } else if (leader) {
                scales[unit] = 0.0f;             // a zero row
            }
        }

        // ---- quantise the second segment (its values are live), rotate the first one again, quantise it
        const float inv = (a32 > 0.0f) ? fminf(__fdividef(7.0f, a32), 3.0e38f) : 0.0f;
        bulk_store_wait_read<0>();           // the store of the previous iteration has read the staging buffer
        __syncwarp();
        const uint32_t tie1 = quantise(v, inv, code_buf + SEG_CODE_BYTES + L.code_lane);
        tok_rotate<LOG2B>(seg_addr, L, v);
        const uint32_t tie0 = quantise(v, inv, code_buf + L.code_lane);
        if (__any_sync(0xffffffffu, (tie0 | tie1) != 0u)) {
            const uint16_t *stage_gen = reinterpret_cast<const uint16_t *>(tsmem + TokSmem::stages);
            const uint16_t *seg = stage_gen + (seg_addr - smem_base - (uint32_t)TokSmem::stages) / 2;
            const uint16_t *raw_row = stage_gen + (row_addr - smem_base - (uint32_t)TokSmem::stages) / 2;
            uint8_t *code_gen = tsmem + TokSmem::codes + (code_buf - smem_base - (uint32_t)TokSmem::codes);
            const uint32_t *xw = reinterpret_cast<const uint32_t *>(tsmem + TokSmem::xch) + (xch_it - smem_base - (uint32_t)TokSmem::xch) / 4;
            __syncwarp();
            if (__any_sync(0xffffffffu, tie0 != 0u))
                tok_fix_ties<LOG2B, MODE, LOG2W>(seg_addr, seg, row_addr, raw_row, xw, code_gen, inv, a32, thr_row, p.sqrt_b, known, a_bits, lane);
            if (__any_sync(0xffffffffu, tie1 != 0u))
                tok_fix_ties<LOG2B, MODE, LOG2W>(seg_addr + SEG_BYTES, seg + SEG_ELEMS, row_addr, raw_row, xw, code_gen + SEG_CODE_BYTES, inv, a32,
                                                 thr_row, p.sqrt_b, known, a_bits, lane);
        }

        // ---- packed codes of both segments: shared staging -> global
        fence_async_smem();
        __syncwarp();
        bulk_store_if(lane == 0, outp, code_buf, TOK_SPW * SEG_CODE_BYTES);
        if (++stage == (uint32_t)NST) { stage = 0; parity ^= 1u; }
    }
    // A load that never completed ends the loop for every warp of the group at the same iteration (they poll
    // the same barrier), so nobody is left behind at the named barrier; the error word tells the host.
    if (lane == 0 && !ok) atomicOr(&g_perq_device_error, 1u);
    if (nreq > 0u) tok_serve_records<LOG2B>(p.x, scales, p.d, p.inv_7_sqrt_b, wreq, nreq, lane);
    bulk_store_wait_read<0>();
}

}  // namespace perq
