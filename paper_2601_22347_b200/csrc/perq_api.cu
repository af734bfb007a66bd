// C ABI of the PeRQ online path: argument validation, kernel selection, launches.
// Nothing here allocates device memory or synchronises, except where perq.h says so.
#include "perq.h"

#include <algorithm>
#include <atomic>
#include <map>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <queue>
#include <utility>
#include <vector>

#include <cuda_runtime.h>
#include <cstring>

#include "perq_generic.cuh"
#include "perq_fast.cuh"
#include "perq_tok.cuh"
#include "perq_mx.cuh"
#include "perq_full.cuh"
#include "perq_stats.cuh"
#include "perq_diag.cuh"
#include "perq_massdiff.cuh"

namespace {

constexpr int kVersion = 100;   // 0.1.0
constexpr size_t kMaxSmem = 227 * 1024;

inline bool is_pow2(long long v) { return v > 0 && (v & (v - 1)) == 0; }
inline int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Order of the base matrix of a b-dimensional Hadamard rotation (Appendix A.1: b = 2^k' * 4t, t the odd part
// of b): 0 for a power of two (Sylvester all the way), 4t when this library has a base matrix of that order
// (Paley's second construction: 4t = 2 (q + 1) with q = 5, 13, 17, 29 or 37), -1 otherwise.
int base_order(int32_t b)
{
    if (b < 1) return -1;
    if (is_pow2(b)) return 0;
    int t = b;
    while ((t & 1) == 0) t >>= 1;
    const int n = 4 * t;
    if (b % n != 0) return -1;
    return (n == 12 || n == 28 || n == 36 || n == 60 || n == 76) ? n : -1;
}

// Rows of the +-1 base matrix of order n = 2 (q + 1) as bit masks (bit c of row r set: entry -1).  Paley's
// second construction: chi = quadratic character mod the prime q = 1 (mod 4); S = symmetric conference matrix
// of order q + 1 (zero corner, ones along the first row and column, chi(i - j) elsewhere); a zero of S becomes
// [[1, -1], [-1, -1]], an entry s = +-1 becomes s [[1, 1], [1, -1]].
void base_matrix_rows(int n, uint32_t (*rows)[3])
{
    const int q = n / 2 - 1;
    int chi[64];
    for (int a = 0; a < q; ++a) chi[a] = -1;
    chi[0] = 0;
    for (int a = 1; a < q; ++a) chi[(a * a) % q] = 1;
    for (int r = 0; r < n; ++r) rows[r][0] = rows[r][1] = rows[r][2] = 0u;
    auto set_neg = [&](int r, int c) { rows[r][c >> 5] |= 1u << (c & 31); };
    for (int i = 0; i <= q; ++i) {
        for (int j = 0; j <= q; ++j) {
            const int sv = (i == 0 && j == 0) ? 0 : (i == 0 || j == 0) ? 1 : chi[((i - j) % q + q) % q];
            const int r = 2 * i, c = 2 * j;
            if (sv == 0) { set_neg(r, c + 1); set_neg(r + 1, c); set_neg(r + 1, c + 1); }
            else if (sv > 0) { set_neg(r + 1, c + 1); }
            else { set_neg(r, c); set_neg(r, c + 1); set_neg(r + 1, c); }
        }
    }
}

// Common shape checks.  On success *g_out is the effective scale-range length.  Block sizes that are not a
// power of two are accepted only where the caller can run them (non_po2_ok) and only as b == d.
int check_shape(int64_t T, int32_t d, int32_t b, int32_t fmt, int32_t group, int *g_out, bool non_po2_ok = false)
{
    if (T < 0 || d <= 0 || d % 32 != 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    if (fmt != PERQ_FMT_INT4 && fmt != PERQ_FMT_MXFP4 && fmt != PERQ_FMT_F32_DEBUG && fmt != PERQ_FMT_FP4 &&
        fmt != PERQ_FMT_INT4_ASYM)
        return PERQ_ERR_FMT;
    if (!is_pow2(b)) {
        if (!non_po2_ok || b != d || base_order(b) <= 0) return PERQ_ERR_BLOCK;
    } else if (b < 16 || b > d || d % b != 0) {
        return PERQ_ERR_BLOCK;
    }
    int g = d;
    if (fmt == PERQ_FMT_INT4) {
        if (group < 0) return PERQ_ERR_GROUP;
        if (group > 0) {
            if (d % group != 0 || group % 8 != 0) return PERQ_ERR_GROUP;
            // a scale range lies inside one Hadamard block or is made of whole blocks: the error bound of a
            // range's maximum is taken from the blocks it covers
            if (group % b != 0 && b % group != 0) return PERQ_ERR_GROUP;
            g = group;
        }
    } else if (fmt == PERQ_FMT_MXFP4) {
        if (group != 0 && group != 32) return PERQ_ERR_GROUP;
        g = 32;
    } else if (fmt == PERQ_FMT_FP4 || fmt == PERQ_FMT_INT4_ASYM) {
        if (group != 0) return PERQ_ERR_GROUP;      // one scale per token
    }
    if (g_out) *g_out = g;
    return PERQ_OK;
}

int sm_count()
{
    static std::atomic<int> cached[64];          // per device ordinal; 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const bool slot = dev >= 0 && dev < 64;
    if (slot && cached[dev].load() > 0) return cached[dev].load();
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (slot) cached[dev].store(n);
    return n;
}

// Opt-in to more than 48 KB of dynamic shared memory.  The attribute belongs to (kernel, device): it is set
// the first time and whenever a launch needs more than was set before (the call costs a microsecond or two,
// which matters for the small launches).
std::mutex g_smem_attr_mutex;
std::map<std::pair<const void *, int>, size_t> g_smem_attr_set;

template <typename K>
int allow_smem(K kernel, size_t bytes)
{
    if (bytes <= 48 * 1024) return PERQ_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PERQ_ERR_CUDA;
    const void *func = reinterpret_cast<const void *>(kernel);
    std::lock_guard<std::mutex> lock(g_smem_attr_mutex);
    size_t &have = g_smem_attr_set[std::make_pair(func, dev)];
    if (have >= bytes) return PERQ_OK;
    if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    have = bytes;
    return PERQ_OK;
}

// Launch with programmatic stream serialization: the kernel may be set up while its predecessor in the stream
// is still running (its prologue overlaps the predecessor's tail); every kernel launched this way calls
// griddep_wait() before its first global memory access, so stream order is kept for all data.
template <typename P>
cudaError_t launch_overlapped(void (*kernel)(P), int grid, int block, size_t smem, cudaStream_t st, const P &params)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, params);
}

int launch_generic(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, int32_t fmt, int g,
                   void *out_codes, void *out_scales, cudaStream_t st)
{
    perq::GenParams p;
    p.x = static_cast<const uint16_t *>(x);
    p.perm = perm;
    p.T = T;
    p.d = d;
    const int n0 = base_order(b);
    if (n0 < 0) return PERQ_ERR_BLOCK;
    p.base_n = n0;
    p.log2b = ilog2(n0 ? b / n0 : b);
    std::memset(p.hrow, 0, sizeof(p.hrow));
    if (n0) base_matrix_rows(n0, p.hrow);
    p.fmt = fmt;
    p.g = g;
    p.out_codes = out_codes;
    p.out_scales = out_scales;
    p.sqrt_b = std::sqrt((double)b);
    p.inv_sqrt_b = (float)(1.0 / p.sqrt_b);
    const perq::GenSmem lay(d, g, p.log2b, n0);
    if (lay.total > kMaxSmem) return PERQ_ERR_SHAPE;
    if (int rc = allow_smem(perq::perq_generic_kernel, lay.total)) return rc;
    const int sms = sm_count();
    if (sms <= 0) return PERQ_ERR_CUDA;
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(2048 / perq::GEN_THREADS, kMaxSmem / lay.total));
    const long long grid = std::min<long long>(T, (long long)sms * per_sm);
    perq::perq_generic_kernel<<<(unsigned)grid, perq::GEN_THREADS, lay.total, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

template <int LOG2B, int MODE, int LOG2G, bool PERM, int XB>
int launch_fast_inst(const perq::FastParams &p, int grid, cudaStream_t st)
{
    auto kernel = perq::perq_fast_kernel<LOG2B, MODE, LOG2G, PERM, XB>;
    const size_t smem = PERM ? perq::FastSmem::total_perm : XB > 3 ? perq::FastSmem::total_full : perq::FastSmem::total;
    if (int rc = allow_smem(kernel, smem)) return rc;
    if (launch_overlapped(kernel, grid, perq::FAST_THREADS, smem, st, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

template <int MODE, int LOG2G, bool PERM>
int launch_fast_b(int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (log2b) {
    case 4: return launch_fast_inst<4, MODE, LOG2G, PERM, 0>(p, grid, st);
    case 5: return launch_fast_inst<5, MODE, LOG2G, PERM, 0>(p, grid, st);
    case 6: return launch_fast_inst<6, MODE, LOG2G, PERM, 0>(p, grid, st);
    default: return launch_fast_inst<7, MODE, LOG2G, PERM, 0>(p, grid, st);
    }
}

template <bool PERM>
int launch_fast_mode(int mode, int G, int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    if (mode == perq::MODE_MX) return launch_fast_b<perq::MODE_MX, 0, PERM>(log2b, p, grid, st);
    if (mode == perq::MODE_G128) return launch_fast_b<perq::MODE_G128, 0, PERM>(log2b, p, grid, st);
    if (mode == perq::MODE_ASYM) {
        switch (G) {
        case 4: return launch_fast_b<perq::MODE_ASYM, 2, PERM>(log2b, p, grid, st);
        case 8: return launch_fast_b<perq::MODE_ASYM, 3, PERM>(log2b, p, grid, st);
        default: return launch_fast_b<perq::MODE_ASYM, -1, PERM>(log2b, p, grid, st);    // G at run time
        }
    }
    if (mode == perq::MODE_FP4) {
        switch (G) {
        case 1: return launch_fast_b<perq::MODE_FP4, 0, PERM>(log2b, p, grid, st);
        case 2: return launch_fast_b<perq::MODE_FP4, 1, PERM>(log2b, p, grid, st);
        case 4: return launch_fast_b<perq::MODE_FP4, 2, PERM>(log2b, p, grid, st);
        case 8: return launch_fast_b<perq::MODE_FP4, 3, PERM>(log2b, p, grid, st);
        default: return launch_fast_b<perq::MODE_FP4, -1, PERM>(log2b, p, grid, st);
        }
    }
    switch (G) {
    case 1: return launch_fast_b<perq::MODE_TOKEN, 0, PERM>(log2b, p, grid, st);
    case 2: return launch_fast_b<perq::MODE_TOKEN, 1, PERM>(log2b, p, grid, st);
    case 4: return launch_fast_b<perq::MODE_TOKEN, 2, PERM>(log2b, p, grid, st);
    case 8: return launch_fast_b<perq::MODE_TOKEN, 3, PERM>(log2b, p, grid, st);
    default: return launch_fast_b<perq::MODE_TOKEN, -1, PERM>(log2b, p, grid, st);   // any other row length: G at run time
    }
}

// full-vector block (b == d): unpermuted, per-token INT4 or MXFP4
template <int MODE>
int launch_fast_full(int G, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (G) {
    case 1: return launch_fast_inst<7, MODE, 0, false, 3>(p, grid, st);
    case 2: return launch_fast_inst<7, MODE, 1, false, 4>(p, grid, st);
    case 4: return launch_fast_inst<7, MODE, 2, false, 5>(p, grid, st);
    default: return launch_fast_inst<7, MODE, 3, false, 6>(p, grid, st);
    }
}

// blocks of 256, 512 or 1024 inside a longer row: unpermuted, per-token INT4 or MXFP4
template <int MODE, int XB>
int launch_fast_long_g(int G, const perq::FastParams &p, int grid, cudaStream_t st)
{
    if (MODE != perq::MODE_TOKEN) return launch_fast_inst<7, MODE, 0, false, XB>(p, grid, st);
    switch (G) {
    case 1: return launch_fast_inst<7, perq::MODE_TOKEN, 0, false, XB>(p, grid, st);
    case 2: return launch_fast_inst<7, perq::MODE_TOKEN, 1, false, XB>(p, grid, st);
    case 4: return launch_fast_inst<7, perq::MODE_TOKEN, 2, false, XB>(p, grid, st);
    default: return launch_fast_inst<7, perq::MODE_TOKEN, 3, false, XB>(p, grid, st);
    }
}

template <int MODE>
int launch_fast_long(int xb, int G, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (xb) {
    case 1: return launch_fast_long_g<MODE, 1>(G, p, grid, st);
    case 2: return launch_fast_long_g<MODE, 2>(G, p, grid, st);
    default: return launch_fast_long_g<MODE, 3>(G, p, grid, st);
    }
}

// Lean MXFP4 kernel: unpermuted, d % 2048 == 0, b <= 128 (a warp's unit is two adjacent segments).
template <int LOG2B>
int launch_mx_inst(const perq::FastParams &p, int grid, cudaStream_t st)
{
    auto kernel = perq::perq_mx_kernel<LOG2B>;
    if (int rc = allow_smem(kernel, perq::MxSmem::total)) return rc;
    if (launch_overlapped(kernel, grid, perq::FAST_THREADS, perq::MxSmem::total, st, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

int launch_mx(int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (log2b) {
    case 4: return launch_mx_inst<4>(p, grid, st);
    case 5: return launch_mx_inst<5>(p, grid, st);
    case 6: return launch_mx_inst<6>(p, grid, st);
    default: return launch_mx_inst<7>(p, grid, st);
    }
}

// Full-vector kernel (b = d = 1024, 2048 or 4096): one round trip through shared memory for the chunk-index bits.
template <int LOG2D, int MODE>
int launch_full_inst(const perq::FastParams &p, int grid, cudaStream_t st)
{
    auto kernel = perq::perq_full_kernel<LOG2D, MODE>;
    if (int rc = allow_smem(kernel, perq::FullSmem::total)) return rc;
    if (launch_overlapped(kernel, grid, perq::FAST_THREADS, perq::FullSmem::total, st, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

template <int MODE>
int launch_full(int segs, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (segs) {
    case 1: return launch_full_inst<10, MODE>(p, grid, st);
    case 2: return launch_full_inst<11, MODE>(p, grid, st);
    default: return launch_full_inst<12, MODE>(p, grid, st);
    }
}

// Lean per-token kernel: INT4 or E2M1 with one scale per token, unpermuted, d in {2048, 4096, 8192}, b <= 128.
template <int LOG2B, int MODE, int LOG2G>
int launch_tok_inst(const perq::FastParams &p, int grid, cudaStream_t st)
{
    auto kernel = perq::perq_tok_kernel<LOG2B, MODE, LOG2G>;
    if (int rc = allow_smem(kernel, perq::TokSmem::total)) return rc;
    if (launch_overlapped(kernel, grid, perq::FAST_THREADS, perq::TokSmem::total, st, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

template <int MODE, int LOG2G>
int launch_tok_b(int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (log2b) {
    case 4: return launch_tok_inst<4, MODE, LOG2G>(p, grid, st);
    case 5: return launch_tok_inst<5, MODE, LOG2G>(p, grid, st);
    case 6: return launch_tok_inst<6, MODE, LOG2G>(p, grid, st);
    default: return launch_tok_inst<7, MODE, LOG2G>(p, grid, st);
    }
}

template <int MODE>
int launch_tok(int segs, int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (segs) {                                      // two segments per warp
    case 2: return launch_tok_b<MODE, 0>(log2b, p, grid, st);
    case 4: return launch_tok_b<MODE, 1>(log2b, p, grid, st);
    default: return launch_tok_b<MODE, 2>(log2b, p, grid, st);
    }
}

// The fast kernel covers d % 1024 == 0 with b <= 128 and scales per token (d / 1024 in {1,2,4,8}),
// per 128 (INT4) or per 32 (MXFP4), with a permutation also d <= 16384; and b == d in {1024 .. 8192}
// without a permutation, per token or MXFP4.  Returns -1 if it does not apply.
int try_launch_fast(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, int32_t fmt, int g,
                    void *out_codes, void *out_scales, cudaStream_t st)
{
    if (d % perq::SEG_ELEMS != 0) return -1;
    const int segs = d / perq::SEG_ELEMS;
    const bool permuted = perm != nullptr;
    const bool full = b == d && b > 128;
    const bool longb = !full && b > 128;                  // 256, 512 or 1024 inside a longer row
    if (longb && (b > perq::SEG_ELEMS || permuted)) return -1;
    if (full && (permuted || (segs != 1 && segs != 2 && segs != 4 && segs != 8))) return -1;
    if (permuted && (d > perq::FastSmem::PERM_MAX_D || segs > perq::FAST_WARPS)) return -1;
    int mode, G = 1;
    if (fmt == PERQ_FMT_MXFP4) {
        mode = perq::MODE_MX;
    } else if (fmt == PERQ_FMT_INT4 && g == 128 && !full && !longb) {
        mode = perq::MODE_G128;
    } else if (fmt == PERQ_FMT_FP4) {
        G = segs;
        if (G > perq::FAST_WARPS - 1 || full || longb) return -1;
        mode = perq::MODE_FP4;
    } else if (fmt == PERQ_FMT_INT4_ASYM) {
        G = segs;
        if (G > perq::FAST_WARPS - 1 || full || longb) return -1;
        mode = perq::MODE_ASYM;
    } else if (fmt == PERQ_FMT_INT4 && g == d) {
        G = segs;
        if (G > perq::FAST_WARPS - 1) return -1;          // named barriers 1..15: one per group of G warps
        if ((full || longb) && G != 1 && G != 2 && G != 4 && G != 8) return -1;
        mode = perq::MODE_TOKEN;
    } else {
        return -1;
    }
    if (permuted || full) G = segs;          // the unit is a whole row
    const long long units = (long long)T * segs / G;
    if (units >= (1ll << 31)) return -1;
    perq::FastParams p;
    p.x = static_cast<const uint16_t *>(x);
    p.out_codes = static_cast<uint8_t *>(out_codes);
    p.out_scales = out_scales;
    p.units_total = (uint32_t)units;
    p.x2 = nullptr;
    p.perm = perm;
    p.G = G;
    p.d = d;
    p.sqrt_b = std::sqrt((double)b);
    p.inv_7_sqrt_b = 1.0 / (7.0 * p.sqrt_b);
    const int sms = sm_count();
    if (sms <= 0) return PERQ_ERR_CUDA;
    const int groups_per_cta = perq::FAST_WARPS / G;
    const long long want = (units + groups_per_cta - 1) / groups_per_cta;
    const int grid = (int)std::min<long long>(want, sms);
    if ((mode == perq::MODE_TOKEN || mode == perq::MODE_FP4) && !permuted && !full && !longb &&
        (segs == 2 || segs == 4 || segs == 8) && b <= 64) {     // (b = 128: the second rotation costs what the sharing saves)
        const int tok_groups = perq::FAST_WARPS / (segs / perq::TOK_SPW);       // rows in flight per CTA
        const int tok_grid = (int)std::min<long long>((T + tok_groups - 1) / tok_groups, sms);
        return mode == perq::MODE_TOKEN ? launch_tok<perq::MODE_TOKEN>(segs, ilog2(b), p, tok_grid, st)
                                        : launch_tok<perq::MODE_FP4>(segs, ilog2(b), p, tok_grid, st);
    }
    if (mode == perq::MODE_MX && !permuted && !full && !longb && segs % perq::MX_SPW == 0) {
        const long long mx_units = (long long)T * segs / perq::MX_SPW;
        p.units_total = (uint32_t)mx_units;
        const int mx_grid = (int)std::min<long long>((mx_units + perq::FAST_WARPS - 1) / perq::FAST_WARPS, sms);
        return launch_mx(ilog2(b), p, mx_grid, st);
    }
    if (full && mode == perq::MODE_MX && segs <= 4)          // (units are rows; grid as computed above)
        return launch_full<perq::MODE_MX>(segs, p, grid, st);
    if (full)
        return mode == perq::MODE_MX ? launch_fast_full<perq::MODE_MX>(G, p, grid, st)
                                     : launch_fast_full<perq::MODE_TOKEN>(G, p, grid, st);
    if (longb)
        return mode == perq::MODE_MX ? launch_fast_long<perq::MODE_MX>(ilog2(b) - 7, G, p, grid, st)
                                     : launch_fast_long<perq::MODE_TOKEN>(ilog2(b) - 7, G, p, grid, st);
    const int log2b = ilog2(b);
    return permuted ? launch_fast_mode<true>(mode, G, log2b, p, grid, st)
                    : launch_fast_mode<false>(mode, G, log2b, p, grid, st);
}

// Gated variants of the group kernel: h = Swish(gate) * up formed in shared memory, then the same path.
template <int LOG2B, int MODE, int LOG2G>
int launch_swiglu_inst(const perq::FastParams &p, int grid, cudaStream_t st)
{
    auto kernel = perq::perq_fast_kernel<LOG2B, MODE, LOG2G, false, 0, true>;
    if (int rc = allow_smem(kernel, perq::FastSmem::total)) return rc;
    if (launch_overlapped(kernel, grid, perq::FAST_THREADS, perq::FastSmem::total, st, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

template <int MODE, int LOG2G>
int launch_swiglu_b(int log2b, const perq::FastParams &p, int grid, cudaStream_t st)
{
    switch (log2b) {
    case 4: return launch_swiglu_inst<4, MODE, LOG2G>(p, grid, st);
    case 5: return launch_swiglu_inst<5, MODE, LOG2G>(p, grid, st);
    case 6: return launch_swiglu_inst<6, MODE, LOG2G>(p, grid, st);
    default: return launch_swiglu_inst<7, MODE, LOG2G>(p, grid, st);
    }
}

int launch_any(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, int32_t fmt, int g,
               void *out_codes, void *out_scales, cudaStream_t st)
{
    if (is_pow2(b)) {
        const int rc = try_launch_fast(x, perm, T, d, b, fmt, g, out_codes, out_scales, st);
        if (rc >= 0) return rc;
    }
    return launch_generic(x, perm, T, d, b, fmt, g, out_codes, out_scales, st);
}

struct StatsPlan {
    int n_cta;
    int rows_per_cta;
    size_t smem;
    size_t ws_bytes;
    int kc;            // 16-byte chunks of a row per thread
    int n_stages;      // stages of the row ring in shared memory
};

template <int KC>
int launch_stats_partial(const perq::StatsParams &p, const struct StatsPlan &plan, cudaStream_t st);

int plan_stats(int64_t T, int32_t d, int32_t b, StatsPlan *plan)
{
    if (T < 0 || d <= 0 || d % 32 != 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    if (!is_pow2(b) || b < 8 || d % b != 0) return PERQ_ERR_BLOCK;
    // The CTA count is a fixed function of the shape (not of the device) so that the
    // order of additions, and with it every output bit, is the same everywhere.
    const int max_cta = 148;
    const long long rows = std::max<long long>(1, (T + max_cta - 1) / max_cta);
    plan->rows_per_cta = (int)std::min<long long>(rows, 1 << 30);
    plan->n_cta = (int)std::max<long long>(1, (T + rows - 1) / rows);
    plan->kc = d <= 4096 ? 1 : d <= 8192 ? 2 : d <= 16384 ? 4 : 8;
    const size_t rpb = 8 / plan->kc;      // rows per batch
    auto smem_for = [&](size_t nst) {
        return nst * rpb * (size_t)d * 2 + (size_t)d * 2 + rpb * (size_t)(d / 8) * 4 + 2 * rpb * 16 * 4 + nst * 8 + 128;
    };
    plan->n_stages = smem_for(3) <= 220 * 1024 ? 3 : 2;
    plan->smem = smem_for((size_t)plan->n_stages);
    plan->ws_bytes = (size_t)plan->n_cta * ((size_t)d + (size_t)(d / b)) * sizeof(float);
    return PERQ_OK;
}

// Scratch of perq_block_l1_stats_static: per-CTA partial sums, resident on every device that
// loads the library.  Each call's first kernel writes every slot its second kernel reads, so
// nothing has to be cleared between calls.
constexpr int kMaxDevices = 64;
static __device__ __align__(256) float g_stats_scratch[PERQ_STATS_STATIC_MAX_FLOATS];
float *g_stats_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_stats_scratch_mutex;

// Per-device resources of perq_rotate_quantize_host's overlap of the two copy directions: one
// non-blocking stream and a few events, created on first use and kept until the process exits.
struct HostPipe {
    static constexpr int kChunks = 4;
    cudaStream_t aux = nullptr;
    cudaEvent_t ready[kChunks] = {};
    cudaEvent_t done = nullptr;
    bool ok = false, tried = false;
};
HostPipe g_host_pipe[kMaxDevices];
std::mutex g_host_pipe_mutex;

HostPipe *host_pipe()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_host_pipe_mutex);
    HostPipe &hp = g_host_pipe[dev];
    if (!hp.tried) {
        hp.tried = true;
        bool ok = cudaStreamCreateWithFlags(&hp.aux, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; ok && i < HostPipe::kChunks; ++i)
            ok = cudaEventCreateWithFlags(&hp.ready[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) (void)cudaGetLastError();
        hp.ok = ok;
    }
    return hp.ok ? &hp : nullptr;     // without it the call still works, on the caller's stream alone
}

template <int KC, int CL, bool WB>
int launch_stats_inst(const perq::StatsParams &p, const StatsPlan &plan, cudaStream_t st)
{
    if (int rc = allow_smem(perq::perq_stats_partial_kernel<KC, CL, WB>, plan.smem)) return rc;
    perq::perq_stats_partial_kernel<KC, CL, WB><<<plan.n_cta, perq::ST_THREADS, plan.smem, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

template <int KC>
int launch_stats_partial(const perq::StatsParams &p, const StatsPlan &plan, cudaStream_t st)
{
    // specialised variants: unpermuted rows of exactly KC * 4096 channels, blocks of 16, 32 or 128
    if (KC <= 4 && p.perm == nullptr && p.d == KC * 4096) {
        const bool wb = p.ws_block != nullptr || p.token_max != nullptr;
        if (!wb) return launch_stats_inst<KC, 2, false>(p, plan, st);
        switch (p.log2b) {
        case 4: return launch_stats_inst<KC, 1, true>(p, plan, st);
        case 5: return launch_stats_inst<KC, 2, true>(p, plan, st);
        case 7: return launch_stats_inst<KC, 4, true>(p, plan, st);
        default: break;
        }
    }
    return launch_stats_inst<KC, -1, false>(p, plan, st);
}

}  // namespace

extern "C" {

int perq_version(void) { return kVersion; }

const char *perq_status_string(int status)
{
    switch (status) {
    case PERQ_OK: return "ok";
    case PERQ_ERR_NULL: return "a required pointer is NULL";
    case PERQ_ERR_SHAPE: return "bad shape: need T >= 0, 0 < d <= 32768, d % 32 == 0 (and the row must fit in shared memory)";
    case PERQ_ERR_BLOCK: return "bad block size: need a power of two b, 16 <= b <= d, dividing d (perq_rotate_quantize also takes b == d = 2^k * 4t with 4t = 12, 28, 36, 60 or 76)";
    case PERQ_ERR_GROUP: return "bad group: INT4 needs 0 or a multiple of 8 that divides d and is a multiple or a divisor of b; MXFP4 needs 0 or 32; FP4 and asymmetric INT4 need 0";
    case PERQ_ERR_FMT: return "unknown format";
    case PERQ_ERR_ALIGN: return "device pointers must be 16-byte aligned";
    case PERQ_ERR_CUDA: return "CUDA runtime error";
    case PERQ_ERR_PERM: return "not a permutation";
    case PERQ_ERR_WORKSPACE: return "workspace missing or too small";
    case PERQ_ERR_UNSUPPORTED: return "combination not covered by this entry point";
    default: return "unknown status";
    }
}

int perq_out_sizes(int64_t T, int32_t d, int32_t fmt, int32_t group, size_t *codes_bytes, size_t *scales_bytes)
{
    if (T < 0 || d <= 0 || d % 32 != 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    size_t cb = 0, sb = 0;
    if (fmt == PERQ_FMT_INT4) {
        if (group < 0 || (group > 0 && (d % group != 0 || group % 8 != 0))) return PERQ_ERR_GROUP;
        cb = (size_t)T * (size_t)(d / 2);
        sb = (size_t)T * (size_t)(group == 0 ? 1 : d / group) * sizeof(float);
    } else if (fmt == PERQ_FMT_MXFP4) {
        if (group != 0 && group != 32) return PERQ_ERR_GROUP;
        cb = (size_t)T * (size_t)(d / 2);
        sb = (size_t)T * (size_t)(d / 32);
    } else if (fmt == PERQ_FMT_FP4 || fmt == PERQ_FMT_INT4_ASYM) {
        if (group != 0) return PERQ_ERR_GROUP;
        cb = (size_t)T * (size_t)(d / 2);
        sb = (size_t)T * sizeof(float) * (fmt == PERQ_FMT_INT4_ASYM ? 2 : 1);
    } else if (fmt == PERQ_FMT_F32_DEBUG) {
        cb = (size_t)T * (size_t)d * sizeof(float);
        sb = 0;
    } else {
        return PERQ_ERR_FMT;
    }
    if (codes_bytes) *codes_bytes = cb;
    if (scales_bytes) *scales_bytes = sb;
    return PERQ_OK;
}

int perq_rotate_quantize(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, int32_t fmt,
                         int32_t group, void *out_codes, void *out_scales, void *stream)
{
    int g = 0;
    if (int rc = check_shape(T, d, b, fmt, group, &g, true)) return rc;
    if (T == 0) return PERQ_OK;   // nothing to read or write: pointers may be anything
    if (!x || !out_codes || (fmt != PERQ_FMT_F32_DEBUG && !out_scales)) return PERQ_ERR_NULL;
    if (!aligned16(x) || !aligned16(out_codes) || !aligned16(out_scales) || !aligned16(perm)) return PERQ_ERR_ALIGN;
    return launch_any(x, perm, T, d, b, fmt, g, out_codes, out_scales, static_cast<cudaStream_t>(stream));
}

int perq_swiglu_rotate_quantize(const void *gate, const void *up, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                                int32_t fmt, int32_t group, void *out_codes, void *out_scales, void *stream)
{
    int g = 0;
    if (int rc = check_shape(T, d, b, fmt, group, &g)) return rc;
    if (perm != nullptr) return PERQ_ERR_UNSUPPORTED;      // in deployment the permutation is merged into the weights
    if (d % perq::SEG_ELEMS != 0 || b > 128) return PERQ_ERR_UNSUPPORTED;
    const int segs = d / perq::SEG_ELEMS;
    int mode, G = 1;
    if (fmt == PERQ_FMT_MXFP4) mode = perq::MODE_MX;
    else if (fmt == PERQ_FMT_INT4 && g == 128) mode = perq::MODE_G128;
    else if (fmt == PERQ_FMT_INT4 && g == d && segs <= perq::FAST_WARPS - 1) { mode = perq::MODE_TOKEN; G = segs; }
    else return PERQ_ERR_UNSUPPORTED;
    if (T == 0) return PERQ_OK;
    if (!gate || !up || !out_codes || !out_scales) return PERQ_ERR_NULL;
    if (!aligned16(gate) || !aligned16(up) || !aligned16(out_codes) || !aligned16(out_scales)) return PERQ_ERR_ALIGN;
    const long long units = (long long)T * segs / G;
    if (units >= (1ll << 31)) return PERQ_ERR_SHAPE;
    perq::FastParams p;
    p.x = static_cast<const uint16_t *>(gate);
    p.x2 = static_cast<const uint16_t *>(up);
    p.out_codes = static_cast<uint8_t *>(out_codes);
    p.out_scales = out_scales;
    p.units_total = (uint32_t)units;
    p.perm = nullptr;
    p.G = G;
    p.d = d;
    p.sqrt_b = std::sqrt((double)b);
    p.inv_7_sqrt_b = 1.0 / (7.0 * p.sqrt_b);
    const int sms = sm_count();
    if (sms <= 0) return PERQ_ERR_CUDA;
    const int groups_per_cta = perq::FAST_WARPS / G;
    const int grid = (int)std::min<long long>((units + groups_per_cta - 1) / groups_per_cta, sms);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int log2b = ilog2(b);
    if (mode == perq::MODE_MX) return launch_swiglu_b<perq::MODE_MX, 0>(log2b, p, grid, st);
    if (mode == perq::MODE_G128) return launch_swiglu_b<perq::MODE_G128, 0>(log2b, p, grid, st);
    return launch_swiglu_b<perq::MODE_TOKEN, -1>(log2b, p, grid, st);       // warps per row at run time
}

int perq_host_workspace_bytes(int64_t T, int32_t d, int32_t fmt, int32_t group, size_t *bytes)
{
    size_t cb = 0, sb = 0;
    if (int rc = perq_out_sizes(T, d, fmt, group, &cb, &sb)) return rc;
    if (!bytes) return PERQ_ERR_NULL;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    *bytes = up((size_t)T * (size_t)d * 2) + up(cb) + up(sb) + 256;
    return PERQ_OK;
}

int perq_rotate_quantize_host(const void *x_host, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                              int32_t fmt, int32_t group, void *out_codes_host, void *out_scales_host,
                              void *workspace, size_t workspace_bytes, void *stream)
{
    int g = 0;
    if (int rc = check_shape(T, d, b, fmt, group, &g, true)) return rc;
    if (T == 0) return PERQ_OK;
    if (!x_host || !out_codes_host || (fmt != PERQ_FMT_F32_DEBUG && !out_scales_host)) return PERQ_ERR_NULL;
    size_t need = 0, cb = 0, sb = 0;
    perq_host_workspace_bytes(T, d, fmt, group, &need);
    perq_out_sizes(T, d, fmt, group, &cb, &sb);
    if (!workspace || workspace_bytes < need) return PERQ_ERR_WORKSPACE;
    if (!aligned16(workspace) || !aligned16(perm)) return PERQ_ERR_ALIGN;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *base = static_cast<unsigned char *>(workspace);
    base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(base) + 255) & ~(uintptr_t)255);
    unsigned char *x_dev = base;
    unsigned char *codes_dev = x_dev + up((size_t)T * (size_t)d * 2);
    unsigned char *scales_dev = codes_dev + up(cb);
    // Rows are independent: larger calls go in four chunks of rows, the copy back of one chunk (on an
    // internal stream) overlapping the copy in of the next, so that both directions of the link are busy.
    HostPipe *pipe = (T >= 4096) ? host_pipe() : nullptr;
    const int n_chunks = pipe ? HostPipe::kChunks : 1;
    const int64_t rows_per = (((T + n_chunks - 1) / n_chunks) + 63) & ~(int64_t)63;
    const size_t code_row = cb / (size_t)T, scale_row = sb / (size_t)T;
    const unsigned char *xh = static_cast<const unsigned char *>(x_host);
    unsigned char *ch = static_cast<unsigned char *>(out_codes_host), *sh = static_cast<unsigned char *>(out_scales_host);
    for (int c = 0; c < n_chunks; ++c) {
        const int64_t r0 = c * rows_per, r1 = std::min<int64_t>(T, r0 + rows_per);
        if (r0 >= r1) break;
        const size_t n = (size_t)(r1 - r0), xo = (size_t)r0 * d * 2, co = (size_t)r0 * code_row, so = (size_t)r0 * scale_row;
        if (cudaMemcpyAsync(x_dev + xo, xh + xo, n * d * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return PERQ_ERR_CUDA;
        if (int rc = launch_any(x_dev + xo, perm, (int64_t)n, d, b, fmt, g, codes_dev + co, scales_dev + so, st)) return rc;
        cudaStream_t back = st;
        if (pipe) {
            if (cudaEventRecord(pipe->ready[c], st) != cudaSuccess || cudaStreamWaitEvent(pipe->aux, pipe->ready[c], 0) != cudaSuccess)
                return PERQ_ERR_CUDA;
            back = pipe->aux;
        }
        if (cudaMemcpyAsync(ch + co, codes_dev + co, n * code_row, cudaMemcpyDeviceToHost, back) != cudaSuccess) return PERQ_ERR_CUDA;
        if (sb && cudaMemcpyAsync(sh + so, scales_dev + so, n * scale_row, cudaMemcpyDeviceToHost, back) != cudaSuccess)
            return PERQ_ERR_CUDA;
    }
    if (pipe && (cudaEventRecord(pipe->done, pipe->aux) != cudaSuccess || cudaStreamWaitEvent(st, pipe->done, 0) != cudaSuccess))
        return PERQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

int perq_block_l1_stats_workspace_bytes(int64_t T, int32_t d, int32_t b, size_t *bytes)
{
    StatsPlan plan;
    if (int rc = plan_stats(T, d, b, &plan)) return rc;
    if (!bytes) return PERQ_ERR_NULL;
    *bytes = plan.ws_bytes;
    return PERQ_OK;
}

int perq_block_l1_stats(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, float *chan_abs_sum,
                        float *block_l1_mean, float *token_max_block_l1, void *workspace, size_t workspace_bytes,
                        void *stream)
{
    StatsPlan plan;
    if (int rc = plan_stats(T, d, b, &plan)) return rc;
    if (!chan_abs_sum && !block_l1_mean && !token_max_block_l1) return PERQ_OK;
    if (!x) return PERQ_ERR_NULL;
    if (T == 0) return PERQ_ERR_SHAPE;
    if (!workspace || workspace_bytes < plan.ws_bytes) return PERQ_ERR_WORKSPACE;
    if (!aligned16(x) || !aligned16(perm) || !aligned16(workspace)) return PERQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    perq::StatsParams p;
    p.x = static_cast<const uint16_t *>(x);
    p.perm = perm;
    p.T = T;
    p.d = d;
    p.log2b = ilog2(b);
    p.rows_per_cta = plan.rows_per_cta;
    p.n_stages = plan.n_stages;
    float *ws = static_cast<float *>(workspace);
    p.ws_chan = chan_abs_sum ? ws : nullptr;
    p.ws_block = block_l1_mean ? ws + (size_t)plan.n_cta * d : nullptr;
    p.token_max = token_max_block_l1;
    int rc = PERQ_OK;
    switch (plan.kc) {
    case 1: rc = launch_stats_partial<1>(p, plan, st); break;
    case 2: rc = launch_stats_partial<2>(p, plan, st); break;
    case 4: rc = launch_stats_partial<4>(p, plan, st); break;
    default: rc = launch_stats_partial<8>(p, plan, st); break;
    }
    if (rc != PERQ_OK) return rc;
    if (chan_abs_sum || block_l1_mean) {
        perq::perq_stats_reduce_kernel<<<(d + 63) / 64, 256, 0, st>>>(
            p.ws_chan, p.ws_block, plan.n_cta, d, d / b, (float)(1.0 / (double)T), chan_abs_sum, block_l1_mean);
        if (cudaGetLastError() != cudaSuccess) return PERQ_ERR_CUDA;
    }
    return PERQ_OK;
}

int perq_block_l1_stats_static(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                                float *chan_abs_sum, float *block_l1_mean, float *token_max_block_l1, void *stream)
{
    StatsPlan plan;
    if (int rc = plan_stats(T, d, b, &plan)) return rc;
    if (plan.ws_bytes > sizeof(g_stats_scratch)) return PERQ_ERR_WORKSPACE;
    if (!chan_abs_sum && !block_l1_mean && !token_max_block_l1) return PERQ_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PERQ_ERR_CUDA;
    float *scratch = nullptr;
    {
        // The array's name is only a host-side handle here; the kernels need its address on
        // the current device, which the runtime hands out per device.
        std::lock_guard<std::mutex> lock(g_stats_scratch_mutex);
        if (g_stats_scratch_addr[dev] == nullptr) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_stats_scratch) != cudaSuccess || p == nullptr) {
                (void)cudaGetLastError();
                return PERQ_ERR_CUDA;
            }
            g_stats_scratch_addr[dev] = static_cast<float *>(p);
        }
        scratch = g_stats_scratch_addr[dev];
    }
    return perq_block_l1_stats(x, perm, T, d, b, chan_abs_sum, block_l1_mean, token_max_block_l1, scratch,
                               sizeof(g_stats_scratch), stream);
}

int perq_token_diagnostics(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b, float *out, void *stream)
{
    if (!x || !out) return PERQ_ERR_NULL;
    if (int rc = check_shape(T, d, b, PERQ_FMT_INT4, 0, nullptr)) return rc;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) != 0 || (reinterpret_cast<uintptr_t>(out) & 3u) != 0 ||
        (perm && (reinterpret_cast<uintptr_t>(perm) & 3u) != 0))
        return PERQ_ERR_ALIGN;
    if (T == 0) return PERQ_OK;
    perq::DiagParams p;
    p.x = static_cast<const uint16_t *>(x);
    p.perm = perm;
    p.out = out;
    p.T = T;
    p.d = d;
    p.log2b = ilog2(b);
    p.inv_sqrt_b = (float)(1.0 / std::sqrt((double)b));
    const perq::DiagSmem lay(d);
    if (lay.total > kMaxSmem) return PERQ_ERR_SHAPE;
    if (int rc = allow_smem(perq::perq_diag_kernel, lay.total)) return rc;
    const int sms = sm_count();
    if (sms <= 0) return PERQ_ERR_CUDA;
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(2048 / perq::GEN_THREADS, kMaxSmem / lay.total));
    const long long grid = std::min<long long>(T, (long long)sms * per_sm);
    perq::perq_diag_kernel<<<(unsigned)grid, perq::GEN_THREADS, lay.total, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

int perq_validate_perm(const int32_t *perm, int32_t d, int32_t *status_dev, void *stream)
{
    if (!perm || !status_dev) return PERQ_ERR_NULL;
    if (d <= 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    const size_t smem = (size_t)((d + 31) / 32) * sizeof(uint32_t);
    perq::perq_validate_perm_kernel<<<1, 1024, smem, static_cast<cudaStream_t>(stream)>>>(perm, d, status_dev);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

int perq_device_error(uint32_t *flags_host)
{
    if (!flags_host) return PERQ_ERR_NULL;
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, perq::g_perq_device_error, sizeof v) != cudaSuccess) return PERQ_ERR_CUDA;
    *flags_host = v;
    return PERQ_OK;
}

int perq_device_error_clear(void)
{
    const unsigned int zero = 0;
    return cudaMemcpyToSymbol(perq::g_perq_device_error, &zero, sizeof zero) == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

int perq_massdiff_perm_device(const float *chan_abs_sum, int32_t d, int32_t b, int32_t *perm, void *workspace,
                              size_t workspace_bytes, void *stream)
{
    if (!chan_abs_sum || !perm) return PERQ_ERR_NULL;
    if (d <= 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    if (b < 1 || d % b != 0 || d / b > perq::MD_MAX_BLOCKS) return PERQ_ERR_BLOCK;
    if (!workspace || workspace_bytes < (size_t)d * sizeof(int32_t)) return PERQ_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(chan_abs_sum) & 3u) != 0 || (reinterpret_cast<uintptr_t>(perm) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(workspace) & 3u) != 0)
        return PERQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *order = static_cast<int32_t *>(workspace);
    perq::perq_massdiff_rank_kernel<<<(d + perq::MD_THREADS - 1) / perq::MD_THREADS, perq::MD_THREADS, 0, st>>>(chan_abs_sum, d, order);
    if (cudaGetLastError() != cudaSuccess) return PERQ_ERR_CUDA;
    perq::perq_massdiff_greedy_kernel<<<1, 32, 0, st>>>(chan_abs_sum, order, d, b, perm);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

int perq_chan_abs_max(const void *x, int64_t T, int32_t d, float *chan_abs_max, void *stream)
{
    if (T < 0 || d <= 0 || d % 32 != 0 || d > PERQ_MAX_D) return PERQ_ERR_SHAPE;
    if (!chan_abs_max || (T > 0 && !x)) return PERQ_ERR_NULL;
    if (!aligned16(x) || (reinterpret_cast<uintptr_t>(chan_abs_max) & 3u) != 0) return PERQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(chan_abs_max, 0, (size_t)d * sizeof(float), st) != cudaSuccess) return PERQ_ERR_CUDA;
    if (T == 0) return PERQ_OK;
    const int col_ctas = (d / 8 + 255) / 256;
    const long long want_slabs = std::max<long long>(1, (4ll * 148 + col_ctas - 1) / col_ctas);
    const long long rows_per = std::max<long long>(8, (T + want_slabs - 1) / want_slabs);
    const long long slabs = (T + rows_per - 1) / rows_per;
    if (slabs > 65535) return PERQ_ERR_SHAPE;
    perq::perq_chan_abs_max_kernel<<<dim3((unsigned)col_ctas, (unsigned)slabs), 256, 0, st>>>(
        static_cast<const uint16_t *>(x), (long long)T, d, (int)rows_per, chan_abs_max);
    return cudaGetLastError() == cudaSuccess ? PERQ_OK : PERQ_ERR_CUDA;
}

namespace {
// channels by descending statistic, equal values by ascending channel
std::vector<int32_t> descending_channels(const float *stat, int32_t d)
{
    std::vector<int32_t> order(d);
    for (int i = 0; i < d; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t l, int32_t r) { return stat[l] > stat[r]; });
    return order;
}
}  // namespace

int perq_absmax_perm(const float *chan_abs_max_host, int32_t d, int32_t *perm_host)
{
    if (!chan_abs_max_host || !perm_host) return PERQ_ERR_NULL;
    if (d <= 0) return PERQ_ERR_SHAPE;
    const std::vector<int32_t> order = descending_channels(chan_abs_max_host, d);
    std::copy(order.begin(), order.end(), perm_host);
    return PERQ_OK;
}

int perq_zigzag_perm(const float *chan_abs_max_host, int32_t d, int32_t b, int32_t *perm_host)
{
    if (!chan_abs_max_host || !perm_host) return PERQ_ERR_NULL;
    if (d <= 0) return PERQ_ERR_SHAPE;
    if (b < 1 || d % b != 0) return PERQ_ERR_BLOCK;
    const std::vector<int32_t> order = descending_channels(chan_abs_max_host, d);
    const int32_t n = d / b;
    for (int32_t r = 0; r < d; ++r) {
        const int32_t round = r / n, pos = r - round * n;
        const int32_t block = (round & 1) ? n - 1 - pos : pos;       // forwards over the blocks, then back
        perm_host[(size_t)block * b + round] = order[r];
    }
    return PERQ_OK;
}

int perq_massdiff_perm(const float *chan_abs_sum_host, int32_t d, int32_t b, int32_t *perm_host)
{
    if (!chan_abs_sum_host || !perm_host) return PERQ_ERR_NULL;
    if (d <= 0) return PERQ_ERR_SHAPE;
    if (b < 1 || d % b != 0) return PERQ_ERR_BLOCK;
    const int n = d / b;
    // channels by descending mass, equal masses by ascending index
    std::vector<int32_t> order(d);
    for (int i = 0; i < d; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t l, int32_t r) {
        return chan_abs_sum_host[l] > chan_abs_sum_host[r];
    });
    // open blocks keyed by (running mass, block index): the top is the lightest, lowest-index block
    using Key = std::pair<double, int32_t>;
    std::priority_queue<Key, std::vector<Key>, std::greater<Key>> open;
    for (int j = 0; j < n; ++j) open.push(Key(0.0, j));
    std::vector<int32_t> fill(n, 0);
    for (int s = 0; s < d; ++s) {
        const int32_t c = order[s];
        Key top = open.top();
        open.pop();
        const int32_t j = top.second;
        perm_host[(size_t)j * b + fill[j]] = c;
        fill[j] += 1;
        if (fill[j] < b) open.push(Key(top.first + (double)chan_abs_sum_host[c], j));
    }
    return PERQ_OK;
}

}  // extern "C"
