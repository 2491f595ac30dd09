// Scale selection, scale sharing and quantization of the multi-scale quantizer in one pass
// (Section "QSGDMaxNormMultiScale Quantization"; Algorithm 2 lines "Compute coordinate scales",
// "Scale sharing" and "Quantize with s*").
//
// With all M workers resident on one GPU the shared index of a coordinate needs no exchange:
// k_i = k(max_m |g^m_i|) (see uq_select.cu).  A thread therefore owns 8 consecutive coordinates of
// ALL workers: it reads the M units once from HBM to form the maximum, finds the 8 shared indices,
// turns them into the 8 factors s_k / W once, and then walks the workers again (their units now
// come from L2) and quantizes each with those factors.  Compared with the selector followed by the
// encoder the gradients cross the HBM interface once instead of twice, the index never comes back
// from memory, and the per-coordinate factor lookup is done once instead of once per worker.
// The results (idx and lev) are bit for bit those of the two separate calls.
#include "uq_device.cuh"
#include "uq_unit.cuh"

namespace uq {

struct SelectEncodeParams {
    const void *g;
    void *lev;
    uint8_t *idx;
    const float *W;
    const int64_t *seg_off;
    uint32_t *status;
    int64_t d, stride, coord0;
    int32_t nseg, M, worker0;
    float cap;                // (float) of the smallest scale: s_hat, the largest level
    ScaleSet scales;
    PhiloxKey key;
};

template <int DT, int FMT, int RNG, int IDXB>
__global__ void __launch_bounds__(kThreads, 3) select_encode_kernel(const __grid_constant__ SelectEncodeParams p)
{
    grid_dependency_prologue();
    using E = Elem<DT>;
    using LF = LevelFmt<FMT>;
    constexpr int H = 8 / E::G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t i = ((int64_t)blockIdx.x * kThreads + tid) * 8;   // my first coordinate
    const int64_t row0 = i - (int64_t)lane * 8;                     // my warp's first coordinate
    if (row0 >= p.d) return;                                        // warp-uniform
    const bool active = i < p.d;
    const char *col = (const char *)p.g + (size_t)i * E::BYTES;

    // pass 1: max over the workers of the magnitude bits (bf16: two coordinates per word)
    uint32_t amag[8];
    if (DT == UQ_F32) {
        float amax[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) amax[e] = 0.0f;
        if (active) {
            int m = 0;
            for (; m + 4 <= p.M; m += 4) {                          // four workers' loads in flight
                uint4 q[4][H];
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int h = 0; h < H; ++h)
                        q[k][h] = ld_stream(col + ((size_t)(m + k) * (size_t)p.stride + h * E::G) * E::BYTES);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float v[8];
#pragma unroll
                    for (int h = 0; h < H; ++h) E::unpack(q[k][h], *(float(*)[E::G])(v + h * E::G));
#pragma unroll
                    for (int e = 0; e < 8; ++e) amax[e] = fmaxf(amax[e], fabsf(v[e]));
                }
            }
            for (; m < p.M; ++m) {
                float v[8];
#pragma unroll
                for (int h = 0; h < H; ++h)
                    E::unpack(ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES),
                              *(float(*)[E::G])(v + h * E::G));
#pragma unroll
                for (int e = 0; e < 8; ++e) amax[e] = fmaxf(amax[e], fabsf(v[e]));
            }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) amag[e] = __float_as_uint(amax[e]);
    } else {
        uint32_t am[4] = {0u, 0u, 0u, 0u};
        if (active) {
            int m = 0;
            for (; m + 8 <= p.M; m += 8) {                          // eight workers' loads in flight
                uint4 q[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) q[k] = ld_stream(col + (size_t)(m + k) * (size_t)p.stride * E::BYTES);
#pragma unroll
                for (int k = 0; k < 8; k += 2) {
                    am[0] = __vimax3_u16x2(am[0], q[k].x & 0x7FFF7FFFu, q[k + 1].x & 0x7FFF7FFFu);
                    am[1] = __vimax3_u16x2(am[1], q[k].y & 0x7FFF7FFFu, q[k + 1].y & 0x7FFF7FFFu);
                    am[2] = __vimax3_u16x2(am[2], q[k].z & 0x7FFF7FFFu, q[k + 1].z & 0x7FFF7FFFu);
                    am[3] = __vimax3_u16x2(am[3], q[k].w & 0x7FFF7FFFu, q[k + 1].w & 0x7FFF7FFFu);
                }
            }
            for (; m < p.M; ++m) {
                const uint4 q = ld_stream(col + (size_t)m * (size_t)p.stride * E::BYTES);
                am[0] = __vmaxu2(am[0], q.x & 0x7FFF7FFFu);
                am[1] = __vmaxu2(am[1], q.y & 0x7FFF7FFFu);
                am[2] = __vmaxu2(am[2], q.z & 0x7FFF7FFFu);
                am[3] = __vmaxu2(am[3], q.w & 0x7FFF7FFFu);
            }
        }
#pragma unroll
        for (int w = 0; w < 4; ++w) { amag[2 * w] = am[w] << 16; amag[2 * w + 1] = am[w] & 0xFFFF0000u; }
    }

    // the shared indices of my 8 coordinates and their factors s_k / W
    __shared__ int32_t sh_thr[kWarps][2 * UQ_MAX_SCALES];
    const int64_t row1 = min(row0 + 256, p.d);
    const int j0 = warp_find_segment(p.seg_off, p.nseg, row0);
    uint64_t packed = 0;
    float inv[8];
    bool overflow = false;
    if (segment_end(p.seg_off, p.nseg, j0, p.d) >= row1) {
        // one segment covers the row: lane k holds the factor and the pass threshold of scale k
        const float inv_lane = inv_scale(p.scales.s[lane & (UQ_MAX_SCALES - 1)], __ldg(p.W + j0));
        overflow = lane < p.scales.N && not_finite(inv_lane);
        sh_thr[warp][lane] = lane < p.scales.N ? pass_threshold(inv_lane, p.cap) : -1;
        __syncwarp();
        const int32_t *T = sh_thr[warp];
        int top = 1;
        while (2 * top < p.scales.N) top *= 2;                      // the bisection's first step
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int32_t a = (int32_t)amag[e];
            int k = 0;
            for (int step = top; step >= 1; step >>= 1)
                if (a <= T[k + step]) k += step;                    // k + step < 2 * top <= 16 + 15
            if (i + e >= p.d) k = 0;                                // padding keeps index 0
            packed |= (uint64_t)k << (e * IDXB);
            inv[e] = __shfl_sync(0xFFFFFFFFu, inv_lane, k);
        }
    } else {
        // a segment boundary crosses the row: the test as written, per coordinate (rare)
        int j = j0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int k = 0;
            inv[e] = 0.0f;
            if (i + e < p.d) {
                j = advance_segment(p.seg_off, p.nseg, j, i + e);
                const float Wj = __ldg(p.W + j), a = __uint_as_float(amag[e]);
                for (int kk = 1; kk < p.scales.N; ++kk)
                    if (__fmul_rn(a, inv_scale(p.scales.s[kk], Wj)) <= p.cap) k = kk;
                inv[e] = inv_scale(p.scales.s[k], Wj);
                overflow |= not_finite(inv[e]);
            }
            packed |= (uint64_t)k << (e * IDXB);
        }
    }
    if (overflow && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
    if (!active) return;
    if (IDXB == 1) p.idx[i >> 3] = (uint8_t)packed;
    else if (IDXB == 2) *(uint16_t *)(p.idx + (i >> 2)) = (uint16_t)packed;
    else if (IDXB == 4) *(uint32_t *)(p.idx + (i >> 1)) = (uint32_t)packed;
    else *(uint64_t *)(p.idx + i) = packed;

    // pass 2: every worker's unit again (from L2 now), quantized with the shared factors
    const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
    const uint32_t blk_lo = (uint32_t)blk, blk_hi = (uint32_t)(blk >> 32);
    const bool ragged = i + 8 > p.d;                                // my unit holds padding
    char *lrow = (char *)p.lev;
    const size_t row_bytes = LF::row_bytes(p.stride);
    // G workers at a time: their loads are in flight together and their Philox chains interleave
#ifdef UQ_FUSED_GROUP
    constexpr int G = UQ_FUSED_GROUP;
#else
    constexpr int G = DT == UQ_BF16 ? 4 : 2;
#endif
    for (int m0 = 0; m0 < p.M; m0 += G) {
        uint4 q[G][H];
#pragma unroll
        for (int n = 0; n < G; ++n) {
            const int m = min(m0 + n, p.M - 1);                     // beyond the last worker: a harmless repeat
#pragma unroll
            for (int h = 0; h < H; ++h) q[n][h] = ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES);
        }
        UnitWords<RNG> rw[G];
        if (RNG == 16) {
            uint32_t wk[G];
            uint4 r[G];
#pragma unroll
            for (int n = 0; n < G; ++n) wk[n] = (uint32_t)(m0 + n + p.worker0);
            philox4x32_10_workers<G>(p.key, blk_lo, blk_hi, wk, r);
#pragma unroll
            for (int n = 0; n < G; ++n) rw[n].r[0] = r[n];
        } else {
#pragma unroll
            for (int n = 0; n < G; ++n) rw[n] = unit_words<RNG>(p.key, blk_lo, blk_hi, (uint32_t)(m0 + n + p.worker0));
        }
#pragma unroll
        for (int n = 0; n < G; ++n) {
            float v[8];
#pragma unroll
            for (int h = 0; h < H; ++h) E::unpack(q[n][h], *(float(*)[E::G])(v + h * E::G));
            if (ragged) {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (i + e >= p.d) v[e] = 0.0f;                  // padding quantizes to level 0
            }
            uint32_t neg_lo, neg_hi;
            unit_signs<DT>(q[n], neg_lo, neg_hi);
            char *row = lrow + (size_t)(m0 + n) * row_bytes;
            quantize_unit_words<FMT, RNG>(v, inv, p.cap, neg_lo, neg_hi, rw[n], row + LF::off(i), row + LF::off2(i, p.stride),
                                          m0 + n < p.M);
        }
    }
}

template <int DT, int FMT, int RNG>
static cudaError_t dispatch_idx(const SelectEncodeParams &p, int idx_bits, cudaStream_t st)
{
    const int64_t blocks = (p.d + kThreads * 8 - 1) / (kThreads * 8);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const unsigned nb = (unsigned)blocks;
    switch (idx_bits) {
    case 1: launch_k(select_encode_kernel<DT, FMT, RNG, 1>, nb, kThreads, st, p); break;
    case 2: launch_k(select_encode_kernel<DT, FMT, RNG, 2>, nb, kThreads, st, p); break;
    case 4: launch_k(select_encode_kernel<DT, FMT, RNG, 4>, nb, kThreads, st, p); break;
    default: launch_k(select_encode_kernel<DT, FMT, RNG, 8>, nb, kThreads, st, p); break;
    }
    return cudaGetLastError();
}

template <int DT>
static cudaError_t dispatch_fmt(const SelectEncodeParams &p, int fmt, int rng_bits, int idx_bits, cudaStream_t st)
{
    switch (fmt) {
    case UQ_FMT_I8:
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I8, 32>(p, idx_bits, st) : dispatch_idx<DT, UQ_FMT_I8, 16>(p, idx_bits, st);
    case UQ_FMT_I4X2:
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I4X2, 32>(p, idx_bits, st) : dispatch_idx<DT, UQ_FMT_I4X2, 16>(p, idx_bits, st);
    case UQ_FMT_I2X4:
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I2X4, 32>(p, idx_bits, st) : dispatch_idx<DT, UQ_FMT_I2X4, 16>(p, idx_bits, st);
    default:
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I6P, 32>(p, idx_bits, st) : dispatch_idx<DT, UQ_FMT_I6P, 16>(p, idx_bits, st);
    }
}

cudaError_t launch_select_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales, int idx_bits,
                                 uint64_t seed, int rng_bits, int fmt, uint8_t *idx, void *lev, uint32_t *status,
                                 cudaStream_t st)
{
    SelectEncodeParams p;
    p.g = g; p.lev = lev; p.idx = idx; p.W = W; p.seg_off = L.seg_off; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.coord0 = L.coord0; p.nseg = L.nseg; p.M = L.M; p.worker0 = L.worker0;
    p.cap = (float)scales.s[0];
    p.scales = scales;
    p.key = philox_key(seed);
    return L.dtype == UQ_F32 ? dispatch_fmt<UQ_F32>(p, fmt, rng_bits, idx_bits, st)
                             : dispatch_fmt<UQ_BF16>(p, fmt, rng_bits, idx_bits, st);
}

}  // namespace uq
