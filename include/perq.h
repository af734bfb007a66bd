/*
 * perq.h -- C ABI of the PeRQ online path for NVIDIA B200 (sm_100a).
 *
 * PeRQ = Permute, Rotate, then Quantize.  For activation rows X[T, d] (bf16) the path is
 *
 *     (X P)  ->  (X P) R~  ->  Q((X P) R~)
 *
 * with P a channel permutation applied as a gather, R~ = I_n (x) R a block-diagonal
 * rotation whose b x b block R is the normalised Sylvester Hadamard matrix, and Q a 4-bit
 * quantiser (symmetric INT4 or MXFP4).  Citations below are to the paper's sections,
 * equations and algorithms.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device memory, "host" pointers ordinary host memory.
 *   - The caller owns every buffer; nothing is allocated, freed or retained by the
 *     library.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream); no call synchronises the device unless it says so.  Outputs are valid
 *     once the caller has synchronised `stream`.
 *   - The return value is a perq_status_t.  Arguments are checked on the host before
 *     anything is launched: on an argument error nothing has been enqueued.  PERQ_ERR_CUDA
 *     (a launch or a copy that the runtime refused) can come after earlier work of the same
 *     call was enqueued: the host-buffer entry point has then already queued its copy to
 *     the device, perq_block_l1_stats its first kernel; the outputs are undefined.
 *   - Device pointers must be 16-byte aligned.  Rows are dense (row stride = d).
 *   - Inputs are assumed finite.  NaN/Inf give unspecified codes but never a fault.
 */
#ifndef PERQ_H
#define PERQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PERQ_FMT_INT4 = 0,      /* symmetric INT4, absmax scale (fp32) per token or per group */
    PERQ_FMT_MXFP4 = 1,     /* E2M1 elements, one E8M0 scale per 32 elements */
    PERQ_FMT_F32_DEBUG = 2, /* no quantisation: the rotated row as fp32 (test hook) */
    PERQ_FMT_FP4 = 3,       /* E2M1 elements, one fp32 scale per token (Appendix B, FP4 activations) */
    PERQ_FMT_INT4_ASYM = 4  /* asymmetric INT4, (scale, zero point) per token (Appendix B, INT4 activations) */
} perq_fmt_t;

typedef enum {
    PERQ_OK = 0,
    PERQ_ERR_NULL = 1,   /* a required pointer is NULL */
    PERQ_ERR_SHAPE = 2,  /* T < 0, d <= 0, d % 32 != 0 or d > PERQ_MAX_D; also: a row that the general kernel cannot
                            hold in 227 KB of shared memory with its per-range tables (very small groups of very long rows) */
    PERQ_ERR_BLOCK = 3,  /* b is neither a power of two in [16, d] that divides d nor (perq_rotate_quantize) a supported b == d = 2^k * 4t */
    PERQ_ERR_GROUP = 4,  /* INT4: group not 0 and (d % group != 0, group % 8 != 0, or group neither a multiple nor a
                            divisor of b); MXFP4: group not 0/32; FP4, INT4_ASYM: not 0 */
    PERQ_ERR_FMT = 5,    /* unknown format */
    PERQ_ERR_ALIGN = 6,  /* a device pointer is not 16-byte aligned */
    PERQ_ERR_CUDA = 7,   /* the CUDA runtime reported an error (launch, copy, attribute) */
    PERQ_ERR_PERM = 8,   /* host-side permutation argument is not a permutation */
    PERQ_ERR_WORKSPACE = 9, /* workspace missing or too small */
    PERQ_ERR_UNSUPPORTED = 10 /* valid arguments that this entry point does not cover (see its description) */
} perq_status_t;

#define PERQ_MAX_D 32768

/*
 * perq_rotate_quantize -- the online hot path, one fused pass.
 *
 * Defined by: Notation paragraph of Sec. 1 (row vector X, d = n*b, block rotation
 * R~ = I_n (x) R, permutation P e_i = e_pi(i)); the block proposition of Sec. 3 and the
 * coordinate form in the proof of the probabilistic proposition (blocks are contiguous
 * index ranges of the permuted row); Sec. 3 for the INT step size
 * s = ||X||_inf / (2^{q-1} - 1); Appendix B for the INT4 and (MX)FP4 quantisers.
 *
 * For every token row t:
 *   1. x'_i = x[t, perm[i]]                       (perm == NULL: x' = x)
 *   2. y_{j*b+i} = b^{-1/2} * sum_{k<b} (-1)^{popcount(i & k)} x'_{j*b+k}   for each block j
 *   3. INT4:  per scale range G (whole row if group == 0, else each `group` consecutive
 *             coordinates of y): a = max_G |y|, s = a / 7, code_i = clip(rne(y_i / s), -8, 7),
 *             stored scale = s as fp32.  a == 0 gives scale 0 and codes 0.
 *      MXFP4: per 32 consecutive coordinates: a = max |y|, E = floor(log2 a) - 2 clamped to
 *             [-127, 127], stored scale byte = E + 127 (0 if a == 0); element code =
 *             sign(y_i) << 3 | index of the nearest of {0, .5, 1, 1.5, 2, 3, 4, 6} to
 *             |y_i| * 2^-E, ties to the even index, saturating at 6.
 *      FP4:   per token: a = max |y|, s = a / 7 (the step the paper gives for FP4 activations), stored as
 *             fp32; element code = sign(y_i) << 3 | index of the nearest of {0, .5, 1, 1.5, 2, 3, 4, 6} to
 *             |y_i| / s, ties to the even index, saturating at 6 (so the row maximum itself saturates).
 *      INT4_ASYM: per token: s = (max y - min y) / 15, z = rne(min y / s),
 *             code_i = clip(rne(y_i / s) - z, 0, 15) (unsigned nibble); the value is s * (code_i + z).
 *             Stored: (s, z) as two fp32.  A constant row gives s = 0, z = 0, codes 0.
 *   4. byte k of the output row = code[2k] | code[2k+1] << 4  (INT4 nibbles are two's complement).
 *
 * x          device, bf16 [T, d] row-major.
 * perm       device, int32 [d], a permutation of 0..d-1, or NULL.  Out-of-range entries
 *            are clamped into range (wrong numbers, never a fault); use
 *            perq_validate_perm to check a permutation beforehand.
 * T, d       rows and channels.  T == 0 is a no-op (pointers are then not looked at).
 *            d % 32 == 0, d <= PERQ_MAX_D.
 * b          a power of two, 16 <= b <= d, with d % b == 0 (b == d is the full-vector rotation); or, for a d
 *            that is not a power of two, b == d = 2^k' * 4t with t the odd part of d and 4t one of 12, 28,
 *            36, 60, 76 (Appendix A.1, "An Optimized Non-Power-of-2 Hadamard Rotation": Llama-3-8B's
 *            14336 = 2^9 * 28, Qwen3's 3072 / 6144 / 12288 = 2^k' * 12 and 9728 = 2^7 * 76).  Step 2 is then
 *            y_i = d^{-1/2} sum_k (-1)^{popcount(floor(i/4t) & floor(k/4t))} B[i mod 4t][k mod 4t] x'_k: rotations
 *            of 4t ADJACENT inputs by a +-1 base matrix B, then k' butterfly stages over strides of 4t.  The
 *            paper does not print its base matrices; B is Paley's second construction for the prime
 *            q = 2t - 1 (symmetric, B B^T = 4t I), so codes need not equal those of another implementation's
 *            matrix.  Other non-power-of-two b, and such a b inside a longer row: PERQ_ERR_BLOCK.
 *            The tensor-core kernels cover d % 1024 == 0 with
 *            b <= 128 (any scale mode, with or without perm) and, unpermuted with per-token or MX
 *            scales, b <= 1024 and b == d <= 8192; everything else runs on a slower general kernel.
 * fmt        perq_fmt_t.
 * group      INT4: 0 (per token) or a multiple of 8 that divides d and is a multiple or a divisor of b.
 *            MXFP4: 0 or 32 (always 32).  FP4, INT4_ASYM: 0.
 *            Scale ranges are consecutive coordinates of the ROTATED row, independent of b.
 * out_codes  device.  INT4/MXFP4: uint8 [T, d/2].  F32_DEBUG: float [T, d] (the rotated row y).
 * out_scales device.  INT4: float [T] or [T, d/group].  MXFP4: uint8 [T, d/32].  FP4: float [T].  INT4_ASYM: float [T, 2].
 *            F32_DEBUG: unused, may be NULL.
 *
 * Codes and scales are deterministic (bit-identical from run to run).  Which kernel serves a call depends
 * on its shape; every kernel stores the fp32 rounding of the exact scale up to one more rounding of a
 * constant factor, so scales of the same row from different shapes' kernels agree to 1 ulp, not bit for bit.
 * Range limit: a token whose largest |y| lies below about 2^-120 (every input subnormal or nearly so) gets
 * the exact scale but all-zero INT4/FP4 codes from the tensor-core kernels, because the fp32 reciprocal of
 * such a scale overflows; the definition would give +-7 at the maximum.
 */
int perq_rotate_quantize(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                         int32_t fmt, int32_t group, void *out_codes, void *out_scales,
                         void *stream);

/*
 * perq_swiglu_rotate_quantize -- the same path fed by the gated activation of a feedforward block.
 *
 * Defined by: the figure on permutation equivariance (the feedforward network of a transformer block):
 * the online rotation's input is h = Swish(x W_gate) (.) (x W_up) -- an elementwise product; Swish(g) =
 * g * sigmoid(g) = g / (1 + exp(-g)) -- and the region is permutation-equivariant, so the permutation is
 * merged into the two projections and none is applied here.  With gate = x W_gate and up = x W_up given as
 * bf16, every row is
 *
 *     h_i = bf16( Swish(gate_i) * up_i )        (the real product, rounded once, to nearest even)
 *
 * followed by steps 2-4 of perq_rotate_quantize on h.  The outputs equal those of perq_rotate_quantize on a
 * materialised h; h is never written to memory (4d + d/2 bytes per token move instead of 8d + d/2).
 * The activation is evaluated in fp32 and again in fp64 wherever the fp32 value is too close to a bf16
 * rounding boundary to decide the rounding, so h is the correctly rounded value.
 *
 * gate, up   device, bf16 [T, d] row-major.      perm   must be NULL (PERQ_ERR_UNSUPPORTED otherwise).
 * Covered:   d % 1024 == 0, b <= 128, and fmt / group = MXFP4, INT4 with group 128, or INT4 per token with
 *            d <= 15360.  Anything else that perq_rotate_quantize would accept returns PERQ_ERR_UNSUPPORTED
 *            (materialise h and call perq_rotate_quantize).
 * Other arguments, outputs and errors as for perq_rotate_quantize.
 */
int perq_swiglu_rotate_quantize(const void *gate, const void *up, const int32_t *perm, int64_t T, int32_t d,
                                int32_t b, int32_t fmt, int32_t group, void *out_codes, void *out_scales,
                                void *stream);

/*
 * perq_out_sizes -- bytes of out_codes and out_scales for a call.  Host only, no CUDA.
 * Either output pointer may be NULL.
 */
int perq_out_sizes(int64_t T, int32_t d, int32_t fmt, int32_t group, size_t *codes_bytes,
                   size_t *scales_bytes);

/*
 * perq_rotate_quantize_host -- the same operation on HOST buffers.
 *
 * Copies x from host memory (pinned memory makes the copies asynchronous), runs
 * perq_rotate_quantize on the device and copies codes and scales back, all on `stream`,
 * then synchronises `stream` before returning.  `workspace` is device memory provided
 * by the caller, at least perq_host_workspace_bytes(...) long; the library allocates
 * nothing.  perm stays a DEVICE pointer (it is reused across calls) or NULL.
 *
 * Calls of 4096 rows or more are processed in four chunks of rows, and the copy back of a
 * chunk runs on an internal non-blocking stream while the next chunk is copied in; that
 * stream and five events are created once per device on first use and kept until exit.
 * Two such calls at the same time on one device (different caller streams) would share
 * those events: issue them from one thread at a time.
 */
int perq_rotate_quantize_host(const void *x_host, const int32_t *perm, int64_t T, int32_t d,
                              int32_t b, int32_t fmt, int32_t group, void *out_codes_host,
                              void *out_scales_host, void *workspace, size_t workspace_bytes,
                              void *stream);
int perq_host_workspace_bytes(int64_t T, int32_t d, int32_t fmt, int32_t group, size_t *bytes);

/*
 * perq_block_l1_stats -- the calibration statistic of the greedy mass-diffusion
 * permutation (Algorithm 1: per-coordinate mean magnitude and per-block mean l1 norm)
 * and of the block proposition's bound ||X R~||_inf <= max_j ||X_{j}||_1 / sqrt(b).
 *
 *   chan_abs_sum[c]       = sum_t |x[t, c]|                         (original channel order)
 *   block_l1_mean[j]      = (1/T) sum_t L[t, j],   L[t, j] = sum_{i<b} |x[t, perm[j*b+i]]|
 *   token_max_block_l1[t] = max_j L[t, j]
 *
 * x, perm, T, d as above (T >= 1 here unless all outputs are NULL); b a power of two
 * >= 8 dividing d.  Each output is device fp32 and may be NULL: [d], [d/b], [T].
 * workspace  device, perq_block_l1_stats_workspace_bytes(...) bytes: per-CTA partial sums
 *            that a second kernel adds in a fixed order, so results are deterministic.
 * Accumulation is fp32: sums agree with exact arithmetic to about 1e-6 relative.
 */
int perq_block_l1_stats(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                        float *chan_abs_sum, float *block_l1_mean, float *token_max_block_l1,
                        void *workspace, size_t workspace_bytes, void *stream);
int perq_block_l1_stats_workspace_bytes(int64_t T, int32_t d, int32_t b, size_t *bytes);

/*
 * perq_block_l1_stats_static -- perq_block_l1_stats for callers that cannot provide a workspace.
 *
 * (No counterpart in the paper: this is a deployment variant of the entry point above.)
 * Some hosts of this library may not allocate device memory at the point where they want
 * the statistic: code that runs inside a memory-pool-managed serving loop whose pool is
 * already fully handed out, plugins that are only given their input and output tensors,
 * or processes whose allocator must stay quiet because allocation would synchronise the
 * device.  For them the per-CTA partial sums go to a fixed array inside the library
 * instead of a caller workspace; outputs and every other argument are as above, and the
 * results are bit-identical to perq_block_l1_stats on the same inputs.
 *
 *   - The array holds PERQ_STATS_STATIC_MAX_FLOATS floats (9.25 MiB) and is part of the
 *     library image: every GPU that loads the library holds it until the process exits.
 *   - A shape is accepted when perq_block_l1_stats_workspace_bytes(T, d, b) fits in the
 *     array, i.e. min(T, 148) * (d + d/b) <= PERQ_STATS_STATIC_MAX_FLOATS; this covers
 *     every d <= 14336 with any T and b >= 8.  Larger shapes return PERQ_ERR_WORKSPACE
 *     and launch nothing.
 *   - The call allocates and frees nothing, on the device or through any library.
 *   - The first call on each device looks up the array's device address (with that
 *     device current) and remembers it; make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to be zero on entry
 *     (each call overwrites what it reads), but two calls whose kernels overlap on the
 *     GPU -- different streams, no ordering between them -- race on it and give wrong
 *     sums.  Calls on one stream, or ordered by events, are safe.
 */
#define PERQ_STATS_STATIC_MAX_FLOATS (148 * 16384)
int perq_block_l1_stats_static(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                               float *chan_abs_sum, float *block_l1_mean,
                               float *token_max_block_l1, void *stream);

/*
 * perq_token_diagnostics -- the per-token quantities the paper plots (the figures on the mass
 * concentration delta, on the block bound versus the block size, and on the bound versus the
 * quantization error), before their normalisation by ||X||_inf.  With x' = gather(x, perm), blocks of
 * b channels, y = x' R~ (block Hadamard rotation) and Q the symmetric 4-bit quantiser of Sec. 3 with one
 * step per token (s = ||y||_inf / 7, round to nearest even), row t of out holds
 *
 *   out[t][0] = ||x||_inf                 out[t][1] = ||x||_1
 *   out[t][2] = max_j ||x'_{j}||_1        (= b max_j delta_{j} ||x'_{j}||_inf, proposition on block rotations)
 *   out[t][3] = ||y||_inf                 out[t][4] = ||y - Q(y)||_2
 *
 * so delta = out1 / (d out0) (proposition on full-vector rotations), the normalised block bound is
 * out2 / (b out0), the outlier suppression ratio out3 / out0, the normalised error out4 / out0.
 *
 *   x, perm, T, d, b   as for perq_rotate_quantize (device pointers; perm may be NULL)
 *   out                float [T, 5], device, written in full; a zero row gives five zeros
 *   stream             cudaStream_t (0 = default); the call only enqueues work
 *
 * Arithmetic is fp32 (sums in a fixed order: outputs are deterministic); the values agree with their
 * real-arithmetic definitions to about 1e-5 relative.  The caller owns every buffer; nothing is
 * allocated.  Errors: as perq_rotate_quantize (NULL, SHAPE, BLOCK, ALIGN, CUDA).
 */
int perq_token_diagnostics(const void *x, const int32_t *perm, int64_t T, int32_t d, int32_t b,
                           float *out, void *stream);

/*
 * perq_validate_perm -- checks on the device that perm[0..d) is a permutation.
 * Writes one int32 to status_dev: 0 = valid, bit 0 = an entry out of range,
 * bit 1 = a duplicate entry.  (Algorithm 1 returns such a permutation; this guards
 * perq_rotate_quantize against a corrupted one.)
 */
int perq_validate_perm(const int32_t *perm, int32_t d, int32_t *status_dev, void *stream);

/*
 * perq_massdiff_perm -- Algorithm 1 (MassDiff), host only, no CUDA.
 *
 * Visits channels in descending chan_abs_sum (ties: lower channel first), assigns each
 * to the not-yet-full block with the smallest running sum (ties: lower block first), and
 * returns the blocks concatenated: perm[j*b + r] = r-th channel assigned to block j.  The
 * result is the `perm` argument of perq_rotate_quantize / perq_block_l1_stats.
 * chan_abs_sum_host: float [d] (e.g. copied back from perq_block_l1_stats; the mean is a
 * positive multiple of the sum, so sums give the same permutation).  perm_host: int32 [d].
 * Running sums are kept in double.  b >= 1, d % b == 0.
 */
int perq_massdiff_perm(const float *chan_abs_sum_host, int32_t d, int32_t b, int32_t *perm_host);

/*
 * perq_chan_abs_max, perq_absmax_perm, perq_zigzag_perm -- the permutations the paper compares MassDiff with
 * (Appendix C, paragraph "Permutations", Table "permute_fn_ablations"; Sec. 4.2 on the zigzag assignment).
 *
 *   perq_chan_abs_max   device: chan_abs_max[c] = max_t |x[t, c]| (float [d], written in full; x bf16 [T, d]
 *                       device, 16-byte aligned; d % 32 == 0).  Enqueues a memset and one kernel on `stream`.
 *   perq_absmax_perm    host only: the channels in descending order of that maximum (equal values: lower
 *                       channel first).
 *   perq_zigzag_perm    host only: the same visiting order dealt to the n = d / b blocks back and forth
 *                       (ranks 0..n-1 to blocks 0..n-1, ranks n..2n-1 to blocks n-1..0, ...); slot r of
 *                       block j holds the channel that round r gave it: perm[j*b + r].
 * The paper prints neither procedure; these are the readings this library takes.  Host arrays: float [d] in,
 * int32 [d] out; the result is a `perm` argument of perq_rotate_quantize / perq_block_l1_stats.
 * Errors: NULL, SHAPE, BLOCK (b < 1 or d % b != 0), ALIGN, CUDA.
 */
int perq_chan_abs_max(const void *x, int64_t T, int32_t d, float *chan_abs_max, void *stream);
int perq_absmax_perm(const float *chan_abs_max_host, int32_t d, int32_t *perm_host);
int perq_zigzag_perm(const float *chan_abs_max_host, int32_t d, int32_t b, int32_t *perm_host);

/*
 * perq_massdiff_perm_device -- Algorithm 1 (MassDiff) on the device: the same permutation as
 * perq_massdiff_perm, entry for entry, from a device array, so that a calibration pass (statistic ->
 * permutation -> permuted rotate+quantize) needs no copy to the host.
 *
 *   chan_abs_sum     float [d], device (e.g. the output of perq_block_l1_stats); finite, non-negative
 *   perm             int32 [d], device, written in full
 *   workspace        device, at least d * 4 bytes (the channels in visiting order); caller-owned
 *   stream           cudaStream_t (0 = default); two kernels are enqueued, nothing is synchronised
 *
 * b >= 1, d % b == 0, d <= PERQ_MAX_D and at most 4096 blocks (d / b).  The greedy is sequential in the
 * channels (one warp scans the open blocks d times): about 2.3 ms for d = 8192, b = 32.
 * Errors: NULL, SHAPE, BLOCK (also: too many blocks), WORKSPACE, ALIGN, CUDA.
 */
int perq_massdiff_perm_device(const float *chan_abs_sum, int32_t d, int32_t b, int32_t *perm,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * perq_device_error -- reads (synchronously, cudaMemcpyFromSymbol) the library's device-side
 * error word on the current device into *flags_host.  0 = no error.  Bit 0 is set when a
 * bounded wait inside a kernel ran out (an asynchronous copy that never completed); the
 * kernel then stops early and its outputs are incomplete.  Kernels only ever set bits; the
 * word keeps them until perq_device_error_clear.
 *
 * perq_device_error_clear -- writes 0 to that word on the current device (synchronously,
 * cudaMemcpyToSymbol), so that a later read reports only what happened since.  Call it with no
 * kernel of the library in flight on the device, or a bit set concurrently may be lost.
 */
int perq_device_error(uint32_t *flags_host);
int perq_device_error_clear(void);

/* Text for a status code (static storage).  Library version = major*10000 + minor*100 + patch. */
const char *perq_status_string(int status);
int perq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PERQ_H */
