/*
 * uq — all-reduce-compatible unbiased gradient quantizers on one B200 (sm_100a).
 *
 * C ABI of the data-parallel hot path of "Unbiased Single-scale and Multi-scale Quantizers for
 * Distributed Optimization": shared max-norm scale -> [per-coordinate scale index] ->
 * stochastic quantization to small integers -> integer sum over workers -> reconstruction of
 * the average gradient (Algorithm 1, QSGDMaxNorm; Algorithm 2, QSGDMaxNormMultiScale).
 *
 * The M workers are M resident device buffers; the paper's three all-reduces (max of the norm,
 * min of the scale index, sum of the levels) are on-device reductions over those buffers.
 *
 * Common rules
 *   - Every data pointer is a DEVICE pointer owned by the caller unless marked "host".
 *     The library allocates no device memory and keeps no state between calls.
 *   - Every call only enqueues kernels on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream) and returns at once; it never synchronizes.
 *   - Return value: UQ_OK or a UQ_ERR_* code.  Argument errors are found on the host before
 *     anything is launched.  Data-dependent problems (non-finite input, a malformed segment
 *     table, s/W overflowing) never trap: the kernels OR a UQ_STATUS_* bit into the caller's
 *     device word `status` (may be NULL to ignore) and still write in-bounds values.
 *   - Layout.  Worker m's gradient is g + m*worker_stride elements, coordinates 0..d-1.
 *     worker_stride is a multiple of 32 and >= d; the padding d..worker_stride-1 of each row
 *     must be readable (its values are ignored).  Level rows use the same stride in coordinates
 *     (int8: worker_stride bytes per row; 4-bit: worker_stride/2 bytes; 2-bit: worker_stride/4 bytes;
 *     6-bit: 3*worker_stride/4 bytes rounded up to 16); the library may write
 *     zeros into a level row's padding.  g and lev must be 16-byte aligned (8-byte rows result for the
 *     2-bit format when worker_stride is not a multiple of 64; that is allowed).
 *   - Segments.  The paper's vector v in R^n is a segment: coordinates seg_off[j]..seg_off[j+1]-1
 *     share the scale W[j].  seg_off is a device array of nseg+1 non-decreasing offsets with
 *     seg_off[0] = 0 and seg_off[nseg] = d; seg_off = NULL (with nseg = 1) means one segment.
 *   - Arithmetic.  Integer results (levels, indices, sums) are defined bit-exactly by the
 *     binary32 operation order stated per call; no fused multiply-add is used where a
 *     floating-point value decides an integer.
 *   - Random draws (the paper's "independent random variables xi_i"): Philox4x32-10 with
 *     key = (seed low, seed high) and counter = (block low, block high, worker, 0), where
 *     worker = layout.worker0 + m is the row's worker number in the whole job.
 *       rng_bits = 32: block = i/4, coordinate i takes word i%4, h = word >> 9 (23 bits)
 *       rng_bits = 16: block = i/8, word (i%8)/2, even i the low half, h = that half (16 bits)
 *     With b the width of h, a coordinate rounds up iff h < rint(p * 2^b) (ties to even), i.e.
 *     with the multiple of 2^-b nearest to the paper's probability p.  i is the coordinate's
 *     index in the worker's whole gradient (layout.coord0 + its index in the buffer).
 *   - Stream order.  The kernels are launched so that the GPU may schedule the blocks of one while
 *     the kernel before it in the stream is still draining (programmatic dependent launch); each
 *     kernel waits for that predecessor to complete before it reads or writes anything, so the
 *     results are those of plain stream order.
 */
#ifndef UQ_H
#define UQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    UQ_OK = 0,
    UQ_ERR_BAD_ARG = 1,     /* null/unaligned pointer, size or parameter out of range */
    UQ_ERR_CUDA = 2,        /* a launch failed; uq_last_cuda_error() has the CUDA code */
    UQ_ERR_UNSUPPORTED = 3, /* a combination this build does not implement */
    UQ_ERR_WORKSPACE = 4    /* workspace too small or missing */
};

enum { UQ_F32 = 0, UQ_BF16 = 1 };              /* gradient element type */
enum { UQ_NORM_LINF = 0, UQ_NORM_L2 = 2 };     /* which norm defines the shared scale */
enum { UQ_FMT_I8 = 0, UQ_FMT_I4X2 = 1, UQ_FMT_I2X4 = 2, UQ_FMT_I6P = 3 }; /* level wire format: 8, 4, 2 or 6 bits per coordinate */
enum { UQ_SRC_LEVELS = 0, UQ_SRC_SUMS = 1 };   /* what uq_decode reads */

/* bits OR-ed into the device status word */
enum {
    UQ_STATUS_NONFINITE = 1,      /* a NaN/Inf input or a non-finite scale */
    UQ_STATUS_BAD_SEGMENTS = 2,   /* seg_off not non-decreasing from 0 to d */
    UQ_STATUS_SCALE_OVERFLOW = 4, /* s / W is not finite (W subnormal-small) */
    UQ_STATUS_BAD_INDEX = 8,      /* a chosen-coordinate index outside [0, d) (uq_randk_*) */
    UQ_STATUS_TIMEOUT = 16        /* a bounded wait inside a kernel ran out (uq_step_small) */
};

#define UQ_MAX_WORKERS 64
#define UQ_MAX_SCALES 16
#define UQ_STATIC_SCRATCH_BYTES (4u << 20) /* scratch built into the library, see uq_agree_scale_static */

typedef struct uq_layout {
    int64_t d;              /* coordinates per worker, >= 0 */
    int64_t worker_stride;  /* coordinates between consecutive workers' rows; multiple of 32, >= d */
    const int64_t *seg_off; /* device, nseg+1 entries, or NULL for a single segment */
    int32_t M;              /* workers, 1..UQ_MAX_WORKERS */
    int32_t nseg;           /* segments, >= 1 */
    int32_t dtype;          /* UQ_F32 or UQ_BF16 (bf16 = upper half of a binary32) */
    int32_t worker0;        /* number, in the whole job, of the worker in row 0 (>= 0); 0 when the
                               buffer holds all workers.  Only the encoders use it: the random
                               draws of row m are those of worker worker0 + m, so a process that
                               holds some of the job's workers produces the same levels */
    int64_t coord0;         /* index, in the worker's whole gradient, of coordinate 0 of this buffer
                               (>= 0, a multiple of 8); 0 when the buffer holds the whole gradient.
                               Only the encoders use it: coordinate i draws the random number of
                               coordinate coord0 + i, so a gradient handed over piece by piece (a
                               bucket at a time, with seg_off counted from the piece's start) gets
                               the levels of the one-piece call */
} uq_layout;

/* Library version (major*10000 + minor*100 + patch). */
int uq_version(void);

/* CUDA error code of the most recent failed launch on the calling thread (0 if none). */
int uq_last_cuda_error(void);

/* Static description of a UQ_ERR_* code. */
const char *uq_error_string(int code);

/* Bytes of device scratch uq_agree_scale needs for this layout (0 on a bad layout). */
size_t uq_workspace_bytes(const uq_layout *layout);

/* Bytes of a packed scale-index stream for this layout: worker_stride * idx_bits / 8. */
size_t uq_index_bytes(const uq_layout *layout, int idx_bits);

/*
 * Shared scale — Algorithm 1 / Algorithm 2, line "MaxAllReduce Norm":
 *   W[j] = max over workers m of || g^m restricted to segment j ||.
 * norm = UQ_NORM_L2 is the paper's definition: every square is formed exactly in binary64,
 * summed in binary64 in a fixed order that does not depend on the launch, and
 * W[j] = (float) sqrt(max_m sum).  norm = UQ_NORM_LINF gives max |g^m_i| exactly.
 * An empty or all-zero segment has W[j] = 0.
 *   g          in   [M][worker_stride] of layout->dtype
 *   W          out  [nseg] float
 *   status     i/o  device word or NULL; NONFINITE if any W[j] is not finite (NaN/Inf input),
 *                   BAD_SEGMENTS if seg_off is malformed (results then unspecified, in bounds)
 *   workspace  scratch of at least uq_workspace_bytes(layout) bytes, 8-byte aligned; contents
 *              need no initialisation and are garbage afterwards
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_WORKSPACE, UQ_ERR_CUDA.
 */
int uq_agree_scale(const uq_layout *layout, const void *g, int norm, float *W, uint32_t *status,
                   void *workspace, size_t workspace_bytes, void *stream);

/*
 * uq_agree_scale for callers that may not allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, not a step of the method.)
 *
 * Who needs it: code that runs where allocation is off limits - a gradient hook invoked while
 * the framework's device allocator must not be entered, a service whose device memory was
 * budgeted and handed out at start-up, a plug-in that only receives the tensors it works on.
 * Such a caller has nowhere to get the scratch buffer that uq_agree_scale asks for, so here
 * the scratch is a fixed array of UQ_STATIC_SCRATCH_BYTES (4 MiB) inside the library image
 * itself.  The cost: every GPU that loads the library carries those 4 MiB until the process
 * exits, whether or not this call is used.
 *
 * Arguments, results and status bits are those of uq_agree_scale without workspace and
 * workspace_bytes; W is bit-identical to what uq_agree_scale writes for the same input.
 *   - Limit: uq_workspace_bytes(layout) must not exceed UQ_STATIC_SCRATCH_BYTES, i.e.
 *     M * (ceil(d / 8192) + nseg) <= 524288 (M = 8 reaches d of about 5e8).  Larger layouts
 *     return UQ_ERR_WORKSPACE and launch nothing; use uq_agree_scale with your own buffer.
 *   - The call itself allocates nothing: no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current) and remembers it; later calls on that
 *     device only launch.  Make that first call during set-up, before any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left
 *     in it.  That is harmless here - every slot is written before it is read, nothing has to
 *     start at zero - but two calls whose kernels overlap on the GPU (different streams, or
 *     different host threads) race on it and produce garbage.  Keep them on one stream, or
 *     order them with events.
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_WORKSPACE (layout too large), UQ_ERR_CUDA.
 */
int uq_agree_scale_static(const uq_layout *layout, const void *g, int norm, float *W, uint32_t *status,
                          void *stream);

/*
 * Single-scale quantizer Q_s — Section "QSGDMaxNorm Quantization" (Eq. Q_s, definition of
 * xi_i), Algorithm 1 line "Quantize gradient", for all M workers:
 *   inv = (float)s / W[j]  (0 if W[j] = 0);  x = min(|v| * inv, (float)s);  l = floor(x);
 *   p = x - l;  level = l + [h < rint(p * 2^b)];  zeta = v < 0 ? -level : level.
 *   lev  out  fmt I8:   int8 [M][worker_stride]               (1 <= s <= 127)
 *             fmt I4X2: two's-complement nibbles, even coordinate in the low nibble,
 *                       [M][worker_stride/2] bytes            (1 <= s <= 7)
 *             fmt I2X4: two's-complement 2-bit fields, coordinate 4q+t in bits 2t..2t+1 of
 *                       byte q, [M][worker_stride/4] bytes    (s = 1: levels -1, 0, 1)
 *             fmt I6P:  two's-complement 6-bit levels in two planes per row: bits 0..3 of every
 *                       level as nibbles (laid out as I4X2) in the first worker_stride/2 bytes,
 *                       bits 4..5 as 2-bit fields (laid out as I2X4) in the worker_stride/4
 *                       bytes after them; rows are 3*worker_stride/4 bytes rounded up to 16
 *                                                              (1 <= s <= 31)
 *   W    in   [nseg], e.g. from uq_agree_scale; any W[j] >= max|v| keeps |zeta| <= s, and
 *             the clamp keeps it so for any W.
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_encode_single(const uq_layout *layout, const void *g, const float *W, int s, uint64_t seed,
                     int rng_bits, int fmt, void *lev, uint32_t *status, void *stream);

/*
 * Per-coordinate scale index with scale sharing — Section "QSGDMaxNormMultiScale
 * Quantization" (the inequality that defines s*_i, and "scale sharing"), Algorithm 2 lines
 * "Compute coordinate scales" and "Scale sharing":
 *   worker's own index  k^m_i = largest k with |g^m_i| * ((float)scales[k] / W[j]) <= (float)scales[0]
 *                       (k = 0 if none; a zero coordinate or W[j] = 0 gives N-1)
 *   shared index        k_i = min over workers of k^m_i.
 *   scales    host  N ascending integers >= 1, N <= UQ_MAX_SCALES; scales[0] is the smallest scale
 *   idx_bits  1 (N <= 2: the two-scale compressors of the paper's experiments), 2 (N <= 4),
 *             4 (N <= 16) or 8
 *   idx       out   packed little-endian within each byte (coordinate i at bit (i*idx_bits)%8
 *                   of byte (i*idx_bits)/8); the buffer holds uq_index_bytes(layout, idx_bits)
 *                   bytes and is 16-byte aligned; the bits of coordinates d .. 8*ceil(d/8)-1
 *                   are written as 0, later bytes are left untouched
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_select_scale_multi(const uq_layout *layout, const void *g, const float *W,
                          const int32_t *scales, int N, int idx_bits, uint8_t *idx,
                          uint32_t *status, void *stream);

/*
 * Multi-scale quantizer Q_{s_} — Section "QSGDMaxNormMultiScale Quantization" (Eq. Q_{s_}),
 * Algorithm 2 line "Quantize with s*": coordinate i of every worker is quantized as in
 * uq_encode_single with s replaced by scales[k_i] in inv and the level clamped to scales[0]
 * (the level fits the bits of the smallest scale).
 *   idx  in  the shared indices written by uq_select_scale_multi (same idx_bits)
 *   fmt  I8 needs scales[0] <= 127, I6P <= 31, I4X2 <= 7, I2X4 needs scales[0] = 1
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_encode_multi(const uq_layout *layout, const void *g, const float *W, const int32_t *scales,
                    int N, const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt,
                    void *lev, uint32_t *status, void *stream);

/*
 * uq_select_encode_multi followed by uq_decode(src = UQ_SRC_LEVELS) as one call — Algorithm 2 from
 * "Compute coordinate scales" to "Reconstruct gradient", everything of a multi-scale step behind
 * the scale agreement.  Where uq_encode_decode is one kernel (int8 levels, 16-bit draws, M <= 8)
 * this is one kernel too: the gradients are read once, the indices, the level rows and the
 * average are written, nothing is read back.  Otherwise the calls it stands for run one after
 * the other.  idx, lev and out receive, bit for bit, what the separate calls write; arguments and
 * errors are theirs.  The first call of this kind on a device (this call, uq_select_encode_multi,
 * or a uq_step that uses them) raises the kernel's limit of dynamic shared memory with
 * cudaFuncSetAttribute before it launches; make that first call during set-up, before any stream
 * capture.  Like uq_select_encode_multi it is bound by instruction issue, not by memory;
 * on a B200 it takes about 19 % less time than uq_select_scale_multi + uq_encode_decode, burst
 * and sustained, which is why uq_step uses it where it is one kernel.
 */
int uq_select_encode_decode_multi(const uq_layout *layout, const void *g, const float *W,
                                  const int32_t *scales, int N, int idx_bits, uint64_t seed, int rng_bits,
                                  int fmt, uint8_t *idx, void *lev, float *out, uint32_t *status,
                                  void *stream);

/*
 * uq_encode_single (scales = NULL) or uq_encode_multi (scales given) followed by
 * uq_decode(src = UQ_SRC_LEVELS) as one call — Algorithm 1 lines "Quantize gradient", "AllReduce
 * gradients", "Reconstruct gradient" (Algorithm 2: "Quantize with s*" onwards) — for callers whose
 * M workers are all in this buffer.  With int8 levels, 16-bit draws and M <= 8 it is one kernel: the
 * CTA that takes a tile of coordinates through the workers adds their levels up in registers and
 * writes the reconstructed average beside the level rows, so the levels are written (they are what
 * would cross the wire) but never read back.  With other formats, more workers or 32-bit draws
 * (whose encoder is bound by its arithmetic: one kernel is then no faster than two) the two kernels
 * run one after the other.  lev and out receive, bit for bit, what the two separate calls write; arguments and
 * errors are theirs (the integer sums are not available here: use uq_decode or uq_aggregate).
 * uq_step makes this call when it is given no S_opt.
 */
int uq_encode_decode(const uq_layout *layout, const void *g, const float *W, int s, const int32_t *scales,
                     int N, const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt,
                     void *lev, float *out, uint32_t *status, void *stream);

/*
 * uq_select_scale_multi followed by uq_encode_multi as one call — Algorithm 2 lines "Compute
 * coordinate scales", "Scale sharing" and "Quantize with s*" — for callers whose M workers are all
 * in this buffer.  With M <= 8 it is one kernel: a CTA copies a tile of every worker's row into
 * shared memory once, takes the maximum over the workers of every magnitude there, finds and stores
 * the shared indices, and quantizes the workers' rows from the same copy, so the gradients cross
 * the memory interface once instead of twice.  With more workers the two kernels run one after
 * the other.  idx and lev receive, bit for bit, what the two separate calls write; arguments and
 * errors are theirs.  On a B200, with bf16 gradients and 16-bit draws, it takes about 15 % less
 * time than the two calls (the gradients are read from memory once); with 32-bit draws, whose
 * encoder is bound by its arithmetic either way, it takes the same time.  It is bound by
 * instruction issue rather than by memory, so uq_step keeps the two streaming kernels and this
 * call is the caller's choice.
 */
int uq_select_encode_multi(const uq_layout *layout, const void *g, const float *W, const int32_t *scales,
                           int N, int idx_bits, uint64_t seed, int rng_bits, int fmt, uint8_t *idx,
                           void *lev, uint32_t *status, void *stream);

/*
 * Integer aggregation — Algorithm 1 / 2 line "AllReduce gradients" without the 1/M:
 *   S[i] = sum over workers of zeta^m_i, in int32.
 *   lev  in   level rows as written by the encoders (layout->dtype is ignored)
 *   S    out  [d] int32, 32-byte aligned (no padding is required or written)
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_aggregate(const uq_layout *layout, const void *lev, int fmt, int32_t *S, void *stream);

/*
 * Reconstruction of the average gradient — Eq. R_s after Algorithm 1 and Eq. R_{s_} after
 * Algorithm 2, applied to the averaged levels:
 *   c = W[j] / ((float)s_i * (float)M);  out[i] = (float)S[i] * c,
 * with s_i = s (scales = NULL) or scales[k_i] (scales, N, idx, idx_bits as in the encoder).
 *   src_kind = UQ_SRC_LEVELS: src is the level rows; the sum over workers and the
 *              reconstruction run fused in one kernel (the sums stay in registers);
 *              S_opt, if not NULL, also receives the int32 sums [d].
 *   src_kind = UQ_SRC_SUMS:   src is int32 S[d] (fmt and S_opt are ignored).
 *   out  [d] float, 32-byte aligned (no padding is required or written); S_opt likewise
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_decode(const uq_layout *layout, const void *src, int src_kind, int fmt, const float *W, int s,
              const int32_t *scales, int N, const uint8_t *idx, int idx_bits, float *out,
              int32_t *S_opt, void *stream);

/*
 * uq_decode(src_kind = UQ_SRC_LEVELS) with the level rows given one by one: lev_rows is a HOST
 * array of layout->M device pointers, lev_rows[m] = start of worker m's level row (16-byte
 * aligned, layout as the encoders write it).  The rows need not lie in one buffer, nor on this
 * GPU: a row in a peer GPU's memory that is mapped into this process (peer access, an IPC or
 * symmetric-memory mapping) is read with ordinary loads over NVLink (on the coherent path, not the
 * read-only one that the one-buffer call uses for its own memory) while it is being summed, so
 * "AllReduce gradients" + "Reconstruct gradient" of Algorithm 1 / 2 run as one kernel that pulls
 * the other workers' levels itself.  The caller orders the call after the peers' encoders (a
 * barrier between the processes); nothing in the kernel waits on another GPU.
 * The array is copied at the call; the other arguments and errors are those of uq_decode.
 */
int uq_decode_rows(const uq_layout *layout, const void *const *lev_rows, int fmt, const float *W, int s,
                   const int32_t *scales, int N, const uint8_t *idx, int idx_bits, float *out,
                   int32_t *S_opt, void *stream);

/*
 * Reconstruction fused with the parameter update — Algorithm 1 / 2, lines "AllReduce gradients",
 * "Reconstruct gradient" and "Update parameters" (theta_{t+1} = theta_t - eta_t * g_hat_t) in one
 * kernel: the level rows are summed and reconstructed as in uq_decode(src = LEVELS) and the
 * result goes from registers into the parameters.  Reading of the optimizer the paper's
 * experiments name (SGD with momentum 0.9 and weight decay 5e-4): per coordinate, in binary32,
 * one IEEE operation per step,
 *   u = g_hat + wd * theta            (skipped when wd == 0)
 *   buf = mu * buf + u;  u = buf      (only when momentum != NULL)
 *   theta = theta - lr * u.
 * momentum = NULL, wd = 0 is the update of Algorithm 1 as printed.
 *   theta     i/o  [d] float, 32-byte aligned, updated in place
 *   momentum  i/o  [d] float, 32-byte aligned, or NULL
 *   out_opt   out  [d] float, 32-byte aligned, or NULL: also receives g_hat
 * scales = NULL selects the single scale s; otherwise scales, N, idx, idx_bits as in the encoder.
 * Errors: UQ_ERR_BAD_ARG (also for NaN lr / mu / wd), UQ_ERR_CUDA.
 */
int uq_decode_update(const uq_layout *layout, const void *lev, int fmt, const float *W, int s,
                     const int32_t *scales, int N, const uint8_t *idx, int idx_bits, float *theta,
                     float *momentum, float lr, float mu, float wd, float *out_opt, void *stream);

/*
 * Scale sharing across processes — Algorithm 2 line "Scale sharing" (s*_i = min over workers)
 * when the M workers are spread over R processes: each process runs uq_select_scale_multi on
 * its own workers (with the job-wide W), the R packed index rows are brought together (an
 * all-gather), and the shared index is their field-wise minimum.
 *   rows      in   [R][row_bytes] packed indices, device, 4-byte aligned, row r = process r
 *   R              1..UQ_MAX_WORKERS
 *   row_bytes      distance between rows, a multiple of 4, >= nbytes
 *   nbytes         bytes of one row to reduce, a multiple of 4 (uq_index_bytes() is one)
 *   idx       out  [nbytes] packed shared indices, 4-byte aligned; may be row 0 of rows
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_CUDA.
 */
int uq_index_min(const uint8_t *rows, int R, int64_t row_bytes, int64_t nbytes, int idx_bits,
                 uint8_t *idx, void *stream);

/*
 * One whole step in one call — Algorithm 1 lines "MaxAllReduce Norm" to "Reconstruct gradient"
 * (scales = NULL: uq_agree_scale, uq_encode_single, uq_decode) or Algorithm 2 (scales given:
 * uq_agree_scale, uq_select_scale_multi, uq_encode_multi, uq_decode), enqueued in that order on
 * `stream`; without S_opt the last two are made as one call, uq_encode_decode, and where that
 * call is one kernel a multi-scale step makes the last three as one, uq_select_encode_decode_multi
 * (two kernels then do the whole step: the norms, and everything else).  Nothing is computed
 * differently: every output is bit for bit that of the separate calls.  Arguments are
 * those of the calls it makes (idx is not used when scales = NULL); the first error stops the
 * sequence and is returned.
 */
int uq_step(const uq_layout *layout, const void *g, int norm, int s, const int32_t *scales, int N,
            int idx_bits, uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev,
            float *out, int32_t *S_opt, uint32_t *status, void *workspace, size_t workspace_bytes,
            void *stream);

/*
 * One whole step as ONE kernel — Algorithm 1 (scales = NULL) or Algorithm 2 (scales given), lines
 * "MaxAllReduce Norm" to "Reconstruct gradient" — for gradients so small that the launches of
 * uq_step cost more than its arithmetic.  A cooperative grid reads the gradients for the norms,
 * meets at one grid-wide barrier, and reads them again (from L2) to [select and share the scale
 * indices,] quantize, store the level rows, add the levels and write the reconstructed average.
 * Arguments as in uq_step.  Supported: one segment (layout->nseg = 1), M <= 8, formats
 * UQ_FMT_I8 / I4X2 / I2X4, both dtypes, norms, draw widths, every index width; worker0 and coord0
 * key the draws as in the encoders.  Anything else returns UQ_ERR_UNSUPPORTED, as does a device
 * without cooperative launches.  Any size is computed correctly; it pays while M * d elements are
 * a few megabytes.
 *   workspace     scratch, device, 8-byte aligned, >= uq_workspace_bytes_small() bytes, used by one
 *                 call at a time.  Its first 64 bytes must be ZERO before the first call (zero
 *                 the scratch once after allocating it); every call leaves them zero again, except
 *                 one that reports UQ_STATUS_TIMEOUT: zero them again after that.
 * Results: idx, lev, S_opt and out are bit for bit those of uq_step given the same W; W is added
 * up in another fixed order (L-inf: identical; L2: within one unit in the last place).
 * The wait at the barrier is bounded: a CTA that gives up sets UQ_STATUS_TIMEOUT and returns
 * (outputs then incomplete).  For that reason status must not be NULL here (UQ_ERR_BAD_ARG).
 * Errors: UQ_ERR_BAD_ARG, UQ_ERR_UNSUPPORTED, UQ_ERR_WORKSPACE, UQ_ERR_CUDA.
 */
size_t uq_workspace_bytes_small(void);
int uq_step_small(const uq_layout *layout, const void *g, int norm, int s, const int32_t *scales, int N,
                  int idx_bits, uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev,
                  float *out, int32_t *S_opt, uint32_t *status, void *workspace, size_t workspace_bytes,
                  void *stream);

/*
 * GlobalRandKMaxNorm / GlobalRandKMaxNormMultiScale — Sections "GlobalRandKMaxNorm Compression"
 * and "GlobalRandKMaxNormMultiScale Compression": every worker keeps the same K coordinates,
 * chosen uniformly at every iteration, and the quantizer of Algorithm 1 / 2 runs on them.
 * The calls below add the choice + gather before, and the scatter after, the dense calls above,
 * which then run on the compact [M][gk_stride] buffer with d = K and one segment.
 *
 * Reading of "choosing K coordinates uniformly": K distinct coordinates sel[t] = pi(t),
 * t = 0..K-1, where pi is a pseudo-random permutation of [0, d) keyed by `seed` (all workers
 * hold the same seed, so they agree without communicating): an alternating Feistel network on
 * b = max(2, ceil(log2 d)) bits (left part b/2 bits; right part the rest; the parts swap each
 * round; new right = old left XOR the low bits of word 0 of Philox4x32-10 with key = seed and
 * counter = (old right, round, 0, 0x4B646E52)), 8 rounds (24 when b < 8), repeated until the
 * value is below d.  No d/K rescaling is applied: the paper states none.
 *
 * uq_randk_gather: sel[t] as above and gk[m][t] = g[m][sel[t]] for every worker.
 *   layout   in   the dense layout of g (d, worker_stride, M, dtype; seg_off / nseg are ignored:
 *                 the K-vector is one vector with one scale)
 *   K             0 <= K <= d
 *   sel      out  [K] int64 device, 8-byte aligned, selection order (not sorted)
 *   gk       out  [M][gk_stride] elements of layout->dtype, 16-byte aligned; gk_stride is a
 *                 multiple of 32 and >= K; elements K .. gk_stride-1 of every row are zeroed
 *   status        UQ_STATUS_BAD_INDEX if a cycle walk did not end within 256 steps
 *                 (probability below 2^-256; the coordinate t is used instead)
 * uq_randk_scatter: out[sel[t]] = vals[t] for t < K; vals = NULL writes zeros (clearing the
 *   entries of an earlier step).  out is [d] float; the other coordinates are not touched.
 * uq_randk_update: theta[sel[t]] = theta[sel[t]] - lr * vals[t] (binary32, product then
 *   difference): Algorithm 1 / 2 line "Update parameters" for a gradient that is zero off the
 *   chosen set.
 *   sel entries outside [0, d) are skipped and set UQ_STATUS_BAD_INDEX; sel must hold distinct
 *   values (as uq_randk_gather writes them), otherwise the result of a repeated entry is
 *   whichever write lands last.
 * Errors: UQ_ERR_BAD_ARG (K outside 0..d, bad stride or alignment, NaN lr), UQ_ERR_CUDA.
 */
int uq_randk_gather(const uq_layout *layout, const void *g, int64_t K, uint64_t seed, int64_t *sel,
                    void *gk, int64_t gk_stride, uint32_t *status, void *stream);
int uq_randk_scatter(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *out,
                     uint32_t *status, void *stream);
int uq_randk_update(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *theta,
                    float lr, uint32_t *status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* UQ_H */
