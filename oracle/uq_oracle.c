/*
 * CPU oracle for the all-reduce-compatible unbiased quantizers
 * (QSGDMaxNorm, Section "QSGDMaxNorm Quantization", Algorithm 1, and
 *  QSGDMaxNormMultiScale, Section "QSGDMaxNormMultiScale Quantization", Algorithm 2).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step statement of what
 * the method computes, used only by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg.  The CUDA library never links, imports or calls it, and it shares no
 * code, header, table or constant generator with the CUDA sources.
 *
 * Conventions
 *   M workers, d coordinates per worker, worker m's vector starts at g + m*stride elements.
 *   Segments j = 0..nseg-1 are the paper's vectors v in R^n: coordinates
 *   seg_off[j] .. seg_off[j+1]-1 share one scale W_j (= ||w||_2 of Algorithm 1).
 *   seg_off == NULL means one segment covering [0, d).
 *   dtype 0 = IEEE binary32, dtype 1 = bfloat16 (upper 16 bits of a binary32).
 *   Window: the per-coordinate functions take coord0 and d and work on the coordinates
 *   coord0 .. coord0+d-1 of the whole vector; their arrays hold just that window (element 0
 *   is coordinate coord0) while seg_off and the random draws keep using whole-vector indices.
 *   coord0 = 0 with d the full length is the ordinary call.
 *
 * Arithmetic: where floating point decides an integer (a level, a scale index) the decision
 * is taken in binary32 with one IEEE operation per written operator; compile with
 * -ffp-contract=off so no multiply-add is fused.  Every function names the passage of the
 * paper it follows; choices the paper leaves open are marked "reading".
 *
 * Pins (tests/test_oracle_*.py): Philox known-answer vectors; closed-form norms; hand-worked
 * examples in exact rational arithmetic (tests/golden); exact-grid inputs; Monte-Carlo
 * unbiasedness and the per-coordinate variance identity from the proof of Lemma 1; the
 * variance bounds of Lemma 1 and Lemma 2; level range; commutation of decode with the sum.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;

/* Number of host threads used by the coordinate loops (1 = serial).  Results do not depend on
 * it: every coordinate is a pure function of its inputs and of a counter-based random draw. */
void uqo_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int uqo_get_threads(void) { return g_threads; }
int uqo_has_openmp(void)
{
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}

/* ------------------------------------------------------------------------------------------
 * Random draws.  The paper only asks for independent random variables xi_i (Eq. for xi in
 * both quantizer sections).  Reading: Philox4x32-10 (Salmon et al., SC'11), a counter-based
 * generator, so that a draw is a pure function of (seed, worker, coordinate).
 * ------------------------------------------------------------------------------------------ */

/* One Philox4x32 block: 10 rounds of two 32x32->64 multiplies and a word permutation;
 * the key is advanced by the two Weyl constants between rounds. */
void uqo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(prod1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)prod1;
        uint32_t n2 = (uint32_t)(prod0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)prod0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The b-bit integer draw h for (seed, worker m, flat coordinate i), 0 <= h < 2^b.
 *   rng_bits == 32: one 32-bit word per coordinate, b = 23 (its upper 23 bits).
 *                   block = i / 4, word = i % 4.
 *   rng_bits == 16: half a word per coordinate, b = 16.
 *                   block = i / 8, word = (i % 8) / 2, even i takes the low half.
 * key = (seed low, seed high); counter = (block low, block high, m, 0).
 * i is the coordinate's index inside the worker's whole d-vector, whatever the segmentation. */
uint32_t uqo_draw(uint64_t seed, uint32_t m, uint64_t i, int rng_bits)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4], out[4];
    if (rng_bits == 32) {
        uint64_t block = i >> 2;
        ctr[0] = (uint32_t)block; ctr[1] = (uint32_t)(block >> 32); ctr[2] = m; ctr[3] = 0;
        uqo_philox4x32_10(ctr, key, out);
        return out[i & 3] >> 9;
    } else {
        uint64_t block = i >> 3;
        ctr[0] = (uint32_t)block; ctr[1] = (uint32_t)(block >> 32); ctr[2] = m; ctr[3] = 0;
        uqo_philox4x32_10(ctr, key, out);
        uint32_t word = out[(i & 7) >> 1];
        return (i & 1) ? (word >> 16) : (word & 0xFFFFu);
    }
}

static int draw_width(int rng_bits) { return rng_bits == 32 ? 23 : 16; }

/* ------------------------------------------------------------------------------------------ */

static float load_elem(const void *g, int dtype, int64_t idx)
{
    if (dtype == 0) return ((const float *)g)[idx];
    uint32_t bits = (uint32_t)((const uint16_t *)g)[idx] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* Segment that holds coordinate i: the j with seg_off[j] <= i < seg_off[j+1]
 * (bisection for the smallest j whose end lies beyond i; empty segments hold nothing). */
static int segment_of(int64_t i, int nseg, const int64_t *seg_off)
{
    if (!seg_off) return 0;
    int lo = 0, hi = nseg - 1;
    while (lo < hi) {
        int mid = (lo + hi) / 2;
        if (seg_off[mid + 1] <= i) lo = mid + 1; else hi = mid;
    }
    return lo;
}

/* ------------------------------------------------------------------------------------------
 * Shared scale, Algorithm 1 line "MaxAllReduce Norm": ||w||_2 = max_m ||g^m||_2, per segment.
 *   norm == 2 : the paper's L2 norm.  Each square is exact in binary64; the sum is carried in
 *               long double in index order; W = (float) sqrt((double) max_m sum).
 *   norm == 0 : L-infinity, W = max_m max_i |g^m_i| (the reading "one shared scale = max|g|"
 *               of the smallest workload).  Both satisfy |v_i| / W <= 1.
 * ------------------------------------------------------------------------------------------ */
void uqo_agree_scale(const void *g, int dtype, int M, int64_t d, int64_t stride, int nseg,
                     const int64_t *seg_off, int norm, float *W)
{
    int64_t whole[2] = { 0, d };
    if (!seg_off) { seg_off = whole; nseg = 1; }
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
    for (int j = 0; j < nseg; ++j) {
        double best = 0.0;
        for (int m = 0; m < M; ++m) {
            long double acc = 0.0L;
            float amax = 0.0f;
            for (int64_t i = seg_off[j]; i < seg_off[j + 1]; ++i) {
                float v = load_elem(g, dtype, (int64_t)m * stride + i);
                if (norm == 2) {
                    double vd = (double)v;
                    acc += (long double)(vd * vd);
                } else {
                    float a = fabsf(v);
                    if (a > amax) amax = a;
                }
            }
            double mine = norm == 2 ? (double)acc : (double)amax;
            if (mine > best) best = mine;
        }
        W[j] = norm == 2 ? (float)sqrt(best) : (float)best;
    }
}

/* s / W in binary32, one division; 0 when the segment is all zeros (then Q(0) = 0). */
static float inv_scale(int32_t s, float W) { return W > 0.0f ? (float)s / W : 0.0f; }

/* ------------------------------------------------------------------------------------------
 * One coordinate of Q_s (Eq. for Q_s and the definition of xi_i that follows it).
 *   a = |v| / W;  reading of the operation order: x = a*s is computed as |v| * (s / W).
 *   l = floor(x) is the paper's l (a in [l/s, (l+1)/s)),  p = x - l is p(a, s) = a*s - l.
 *   xi = (l+1)/s with probability p, else l/s.  Reading: with a b-bit draw h the probability is
 *   the multiple of 2^-b nearest to p: round up iff h < rint(p * 2^b) (ties to even).
 *   a = 1 has no l < s; reading: x is clamped to s, giving level s with p = 0.
 *   Returned: zeta_i = sign(v) * s * xi_i, an integer in [-s_cap, s_cap].
 * ------------------------------------------------------------------------------------------ */
static int quantize_coord(float v, float inv, float s_cap, uint32_t h, int b)
{
    float x = fabsf(v) * inv;
    if (!(x <= s_cap)) x = s_cap;
    float l = floorf(x);
    float p = x - l;
    float threshold = rintf(ldexpf(p, b));
    int up = (float)h < threshold;
    int level = (int)l + up;
    return v < 0.0f ? -level : level;
}

/* Algorithm 1 line "Quantize gradient" for every worker: zeta^m = Q_s(g^m, ||w||_2).
 * lev[m*stride + i] receives zeta^m_i as int8 (s <= 127).
 * h_inject != NULL replaces the Philox draw of coordinate (m, i) by h_inject[m*stride + i]
 * (used by the worked examples).
 * worker0: the rows of g are workers worker0 .. worker0+M-1 of the whole job (a process that
 * holds only some of the M workers passes its first worker's number; the draws are keyed by
 * the worker's number in the job, so the levels do not depend on who computes them). */
void uqo_encode_single(const void *g, int dtype, int M, int64_t coord0, int64_t d, int64_t stride,
                       int nseg, const int64_t *seg_off, const float *W, int32_t s,
                       uint64_t seed, int rng_bits, const uint32_t *h_inject, int8_t *lev, int worker0)
{
    int b = draw_width(rng_bits);
    for (int m = 0; m < M; ++m) {
#pragma omp parallel for schedule(static) num_threads(g_threads)
        for (int64_t i = 0; i < d; ++i) {
            int j = segment_of(coord0 + i, nseg, seg_off);
            float inv = inv_scale(s, W[j]);
            float v = load_elem(g, dtype, (int64_t)m * stride + i);
            uint32_t h = h_inject ? h_inject[(int64_t)m * stride + i]
                                  : uqo_draw(seed, (uint32_t)(worker0 + m), (uint64_t)(coord0 + i), rng_bits);
            lev[(int64_t)m * stride + i] = (int8_t)quantize_coord(v, inv, (float)s, h, b);
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 2 lines "Compute coordinate scales" and "Scale sharing".
 * Worker m's own scale for coordinate i is the largest s in the scale set with
 *   s <= (||w||_2 / |v_i|) * min_j s_j           (the displayed inequality after Q_{s_}),
 * tested as |v_i| * (s_k / W) <= s_hat in binary32 (reading: multiply through by |v_i|/W so
 * that v_i = 0 needs no division; equality counts; if no scale passes, the smallest is used).
 * The shared index is the minimum over workers.  scales[] is ascending, s_hat = scales[0].
 * idx[i] receives the shared index k_i (one byte per coordinate);
 * own != NULL also receives each worker's own index at own[m*stride + i].
 * ------------------------------------------------------------------------------------------ */
void uqo_select_scale_multi(const void *g, int dtype, int M, int64_t coord0, int64_t d,
                            int64_t stride, int nseg, const int64_t *seg_off, const float *W,
                            const int32_t *scales, int N, uint8_t *idx, uint8_t *own)
{
    float s_hat = (float)scales[0];
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int64_t i = 0; i < d; ++i) {
        int j = segment_of(coord0 + i, nseg, seg_off);
        int shared = N - 1;
        for (int m = 0; m < M; ++m) {
            float v = load_elem(g, dtype, (int64_t)m * stride + i);
            int mine = 0;
            for (int k = 0; k < N; ++k) {
                float xk = fabsf(v) * inv_scale(scales[k], W[j]);
                if (xk <= s_hat) mine = k;
            }
            if (own) own[(int64_t)m * stride + i] = (uint8_t)mine;
            if (mine < shared) shared = mine;
        }
        idx[i] = (uint8_t)shared;
    }
}

/* Algorithm 2 line "Quantize with s*": coordinate i of every worker is quantized by Q_s with
 * s = scales[idx[i]]; the level is representable in the bits of the smallest scale, so it is
 * clamped to s_hat = scales[0]. */
void uqo_encode_multi(const void *g, int dtype, int M, int64_t coord0, int64_t d, int64_t stride,
                      int nseg, const int64_t *seg_off, const float *W, const int32_t *scales,
                      int N, const uint8_t *idx, uint64_t seed, int rng_bits,
                      const uint32_t *h_inject, int8_t *lev, int worker0)
{
    int b = draw_width(rng_bits);
    float s_hat = (float)scales[0];
    (void)N;
    for (int m = 0; m < M; ++m) {
#pragma omp parallel for schedule(static) num_threads(g_threads)
        for (int64_t i = 0; i < d; ++i) {
            int j = segment_of(coord0 + i, nseg, seg_off);
            float inv = inv_scale(scales[idx[i]], W[j]);
            float v = load_elem(g, dtype, (int64_t)m * stride + i);
            uint32_t h = h_inject ? h_inject[(int64_t)m * stride + i]
                                  : uqo_draw(seed, (uint32_t)(worker0 + m), (uint64_t)(coord0 + i), rng_bits);
            lev[(int64_t)m * stride + i] = (int8_t)quantize_coord(v, inv, s_hat, h, b);
        }
    }
}

/* Algorithm 1/2 line "AllReduce gradients", the integer part: S_i = sum_m zeta^m_i.
 * Reading: the accumulator is int32 (|S_i| <= M * 127). */
void uqo_aggregate(const int8_t *lev, int M, int64_t d, int64_t stride, int32_t *S)
{
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int64_t i = 0; i < d; ++i) {
        int32_t acc = 0;
        for (int m = 0; m < M; ++m) acc += lev[(int64_t)m * stride + i];
        S[i] = acc;
    }
}

/* Reconstruction R_s (Eq. after Algorithm 1) and R_{s_} (Eq. after Algorithm 2) applied to
 * the averaged levels zeta = S / M:   g_hat_i = W_j * S_i / (s_i * M).
 * Reading of the operation order: c = W_j / ((float)s_i * (float)M), g_hat_i = (float)S_i * c.
 * scales == NULL: single scale s.  Otherwise s_i = scales[idx[i]]. */
void uqo_decode(const int32_t *S, int M, int64_t coord0, int64_t d, int nseg,
                const int64_t *seg_off,
                const float *W, int32_t s, const int32_t *scales, const uint8_t *idx,
                float *out)
{
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int64_t i = 0; i < d; ++i) {
        int j = segment_of(coord0 + i, nseg, seg_off);
        int32_t si = scales ? scales[idx[i]] : s;
        float c = W[j] / ((float)si * (float)M);
        out[i] = (float)S[i] * c;
    }
}

/* The same reconstruction in binary64 (for the commutation pin: decode of the sum versus the
 * mean of per-worker decodes). */
void uqo_decode_f64(const int32_t *S, int M, int64_t coord0, int64_t d, int nseg,
                    const int64_t *seg_off,
                    const float *W, int32_t s, const int32_t *scales, const uint8_t *idx,
                    double *out)
{
    for (int64_t i = 0; i < d; ++i) {
        int j = segment_of(coord0 + i, nseg, seg_off);
        int32_t si = scales ? scales[idx[i]] : s;
        out[i] = (double)W[j] * (double)S[i] / ((double)si * (double)M);
    }
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1 / 2, line "Update parameters": theta_{t+1} = theta_t - eta_t * g_hat_t.
 * Reading of the optimizer named in Section "Experiments" (SGD, momentum mu, weight decay wd):
 *   u = g_hat + wd * theta;  buf = mu * buf + u, u = buf (if a momentum buffer is given);
 *   theta = theta - lr * u.       mom == NULL, wd = 0 is the printed update.
 * Binary32, one IEEE operation per written operator (the weight-decay term is skipped when
 * wd == 0, so that the printed update is exactly theta - lr * g_hat).
 * ------------------------------------------------------------------------------------------ */
void uqo_sgd_update(const float *g_hat, int64_t d, float *theta, float *mom, float lr, float mu, float wd)
{
    for (int64_t i = 0; i < d; ++i) {
        float u = g_hat[i];
        if (wd != 0.0f) { float t = wd * theta[i]; u = u + t; }
        if (mom) { float t = mu * mom[i]; mom[i] = t + u; u = mom[i]; }
        float step = lr * u;
        theta[i] = theta[i] - step;
    }
}

/* ------------------------------------------------------------------------------------------
 * Wire formats (the bit counts r = ceil(log s) + 1 and + ceil(log N) of the two sections).
 * ------------------------------------------------------------------------------------------ */

/* 4-bit levels (s <= 7): two's-complement nibbles, even coordinate in the low nibble;
 * packed[m*stride/2 + q] holds coordinates 2q and 2q+1 of worker m; an odd tail has a zero
 * high nibble. */
void uqo_pack_levels_i4(const int8_t *lev, int M, int64_t d, int64_t stride, uint8_t *packed)
{
    for (int m = 0; m < M; ++m)
        for (int64_t q = 0; 2 * q < d; ++q) {
            int lo = lev[(int64_t)m * stride + 2 * q];
            int hi = 2 * q + 1 < d ? lev[(int64_t)m * stride + 2 * q + 1] : 0;
            packed[(int64_t)m * (stride / 2) + q] = (uint8_t)((lo & 15) | ((hi & 15) << 4));
        }
}

/* 2-bit levels (s = 1, zeta in {-1, 0, 1}): two's-complement 2-bit fields, four coordinates per
 * byte, coordinate 4q+t in bits 2t..2t+1; packed[m*stride/4 + q]; fields beyond d are zero. */
void uqo_pack_levels_i2(const int8_t *lev, int M, int64_t d, int64_t stride, uint8_t *packed)
{
    for (int m = 0; m < M; ++m)
        for (int64_t q = 0; 4 * q < d; ++q) {
            unsigned byte = 0;
            for (int t = 0; t < 4; ++t) {
                int64_t i = 4 * q + t;
                if (i < d) byte |= ((unsigned)lev[(int64_t)m * stride + i] & 3u) << (2 * t);
            }
            packed[(int64_t)m * (stride / 4) + q] = (uint8_t)byte;
        }
}

/* 6-bit levels (s <= 31) in two planes per row: bits 0..3 of the two's-complement level as
 * nibbles (even coordinate in the low nibble) in the first stride/2 bytes of the row, bits 4..5
 * as 2-bit fields (coordinate 4q+t in bits 2t..2t+1 of byte q) in the stride/4 bytes after
 * them (stride = the layout's row stride in coordinates); rows are row_bytes apart; everything
 * else in a row is zero. */
void uqo_pack_levels_i6p(const int8_t *lev, int M, int64_t d, int64_t lev_stride, int64_t stride, int64_t row_bytes,
                         uint8_t *packed)
{
    memset(packed, 0, (size_t)M * (size_t)row_bytes);
    for (int m = 0; m < M; ++m)
        for (int64_t i = 0; i < d; ++i) {
            const unsigned u = (unsigned)lev[(int64_t)m * lev_stride + i] & 63u;     /* lev rows are lev_stride apart */
            uint8_t *row = packed + (int64_t)m * row_bytes;
            row[i / 2] |= (uint8_t)((u & 15u) << (4 * (i % 2)));
            row[stride / 2 + i / 4] |= (uint8_t)((u >> 4) << (2 * (i % 4)));
        }
}

/* Scale sharing across processes (Algorithm 2 line "Scale sharing" when each process holds
 * some of the workers): rows[r*d + i] is the minimum over process r's workers, the shared
 * index is the minimum over the R rows. */
void uqo_index_min(const uint8_t *rows, int R, int64_t d, uint8_t *idx)
{
    for (int64_t i = 0; i < d; ++i) {
        uint8_t k = rows[i];
        for (int r = 1; r < R; ++r)
            if (rows[(int64_t)r * d + i] < k) k = rows[(int64_t)r * d + i];
        idx[i] = k;
    }
}

/* Scale indices packed idx_bits (2, 4 or 8) per coordinate, little-endian inside the byte:
 * coordinate i sits at bit (i * idx_bits) % 8 of byte (i * idx_bits) / 8; unused tail bits 0. */
void uqo_pack_index(const uint8_t *idx, int64_t d, int idx_bits, uint8_t *packed)
{
    int per = 8 / idx_bits;
    int64_t nbytes = (d + per - 1) / per;
    for (int64_t q = 0; q < nbytes; ++q) {
        unsigned byte = 0;
        for (int t = 0; t < per; ++t) {
            int64_t i = q * per + t;
            if (i < d) byte |= (unsigned)idx[i] << (t * idx_bits);
        }
        packed[q] = (uint8_t)byte;
    }
}

/* ------------------------------------------------------------------------------------------
 * GlobalRandKMaxNorm / GlobalRandKMaxNormMultiScale (Sections "GlobalRandKMaxNorm Compression"
 * and "GlobalRandKMaxNormMultiScale Compression"): every worker keeps the same K coordinates,
 * chosen uniformly, and the quantizer of Algorithm 1 / 2 runs on the K-vector.
 *
 * Reading (the paper says only "choosing K coordinates uniformly"): the K coordinates are
 * distinct; they are sel[t] = pi(t), t = 0..K-1, for a pseudo-random permutation pi of
 * [0, d) keyed by the shared seed, so all workers agree without communicating.  pi is an
 * alternating Feistel network on b = max(2, ceil(log2 d)) bits whose round function is a
 * Philox4x32-10 word, restricted to [0, d) by cycle walking (apply the network until the
 * value is below d; 2^b < 2d, so a step leaves the range with probability < 1/2).  The
 * network has 8 rounds, 24 when b < 8: round functions of one to three bits carry so little
 * randomness that a short network visibly favours some orderings of a tiny domain.
 * No rescaling by d/K: the paper states none.
 * ------------------------------------------------------------------------------------------ */
static uint64_t randk_network(uint64_t x, int b, uint64_t seed)
{
    int a = b / 2, c = b - a;                         /* widths of the left and right part */
    uint64_t L = x >> c, R = x & (((uint64_t)1 << c) - 1);
    const uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    const uint32_t rounds = b < 8 ? 24u : 8u;
    for (uint32_t r = 0; r < rounds; ++r) {
        /* counter word 3 is a tag that the rounding draws (which use 0 there) never use */
        const uint32_t ctr[4] = { (uint32_t)R, r, 0u, 0x4B646E52u };
        uint32_t out[4];
        uqo_philox4x32_10(ctr, key, out);
        const uint64_t newR = L ^ ((uint64_t)out[0] & (((uint64_t)1 << a) - 1));
        L = R; R = newR;                              /* the parts swap, and so do their widths */
        const int t = a; a = c; c = t;
    }
    return (L << c) | R;                              /* an even number of rounds: the widths are back in place */
}

void uqo_randk_indices(int64_t d, int64_t K, uint64_t seed, int64_t *sel)
{
    int b = 2;
    while (((int64_t)1 << b) < d) ++b;
    for (int64_t t = 0; t < K; ++t) {
        uint64_t x = (uint64_t)t;
        do x = randk_network(x, b, seed); while (x >= (uint64_t)d);
        sel[t] = (int64_t)x;
    }
}

/* gk[m][t] = g[m][sel[t]]; elements t = K .. strideK-1 of every row are zero. */
void uqo_randk_gather(const void *g, int dtype, int M, int64_t stride, int64_t K, const int64_t *sel,
                      void *gk, int64_t strideK)
{
    const size_t eb = dtype == 0 ? 4 : 2;
    memset(gk, 0, (size_t)M * (size_t)strideK * eb);
    for (int m = 0; m < M; ++m)
        for (int64_t t = 0; t < K; ++t)
            memcpy((char *)gk + ((size_t)m * (size_t)strideK + (size_t)t) * eb,
                   (const char *)g + ((size_t)m * (size_t)stride + (size_t)sel[t]) * eb, eb);
}

/* out[sel[t]] = vals[t] (vals == NULL: 0), the other coordinates of out are left alone. */
void uqo_randk_scatter(int64_t K, const int64_t *sel, const float *vals, float *out)
{
    for (int64_t t = 0; t < K; ++t) out[sel[t]] = vals ? vals[t] : 0.0f;
}

/* Algorithm 1 / 2, line "Update parameters", with a gradient that is zero off the chosen set:
 * theta[sel[t]] -= lr * vals[t] (binary32, product then difference). */
void uqo_randk_update(int64_t K, const int64_t *sel, const float *vals, float *theta, float lr)
{
    for (int64_t t = 0; t < K; ++t) {
        const float step = lr * vals[t];
        theta[sel[t]] = theta[sel[t]] - step;
    }
}
