// Stochastic quantization of every worker's gradient to small signed integers:
// Q_s (Section "QSGDMaxNorm Quantization", Algorithm 1 line "Quantize gradient") and
// Q_{s_} with the shared per-coordinate scale (Section "QSGDMaxNormMultiScale Quantization",
// Algorithm 2 line "Quantize with s*").
//
// One streaming pass: a thread owns units of 8 consecutive coordinates (32 B of fp32 or 16 B of
// bf16 in, 8 B of int8 or 4 B of packed 4-bit levels out); a CTA owns one tile of one worker.
// A worker's CTA reads only that worker's gradient plus the agreed values W and idx.
#include "uq_device.cuh"

namespace uq {

struct EncodeParams {
    const void *g;
    void *lev;
    const float *W;
    const int64_t *seg_off;
    const uint8_t *idx;
    uint32_t *status;
    int64_t d, stride;
    uint64_t seed;
    int32_t nseg, M;
    float cap;                // (float) of the smallest scale: the largest level
    ScaleSet scales;          // single-scale: N = 1, s[0] = s
};

template <int DT> struct EncodeShape {
    static constexpr int UNITS = DT == UQ_F32 ? 2 : 4;          // 64 B of input per thread
    static constexpr int TILE = kThreads * UNITS * 8;
};

// (float)s_k / W with one IEEE division; 0 for an all-zero segment.
__device__ __forceinline__ float inv_scale(int32_t s, float W)
{
    return W > 0.0f ? __fdiv_rn((float)s, W) : 0.0f;
}

template <int IDXB> __device__ __forceinline__ uint64_t load_idx8(const uint8_t *idx, int64_t i)
{
    // the idx_bits * 8 bits that belong to coordinates i..i+7 (i is a multiple of 8)
    if (IDXB == 2) return *(const uint16_t *)(idx + (i >> 2));
    if (IDXB == 4) return *(const uint32_t *)(idx + (i >> 1));
    return *(const uint64_t *)(idx + i);
}

template <int DT, int FMT, int RNG, int IDXB>
__global__ void __launch_bounds__(kThreads) encode_kernel(const EncodeParams p)
{
    using E = Elem<DT>;
    using S = EncodeShape<DT>;
    constexpr bool MULTI = IDXB != 0;
    const int m = blockIdx.x % p.M;
    const int64_t tile = blockIdx.x / p.M;
    const int64_t t0 = tile * S::TILE;
    const int64_t t1 = min(t0 + (int64_t)S::TILE, p.d);
    const int tid = threadIdx.x;
    const char *row = (const char *)p.g + (size_t)m * (size_t)p.stride * E::BYTES;

    // issue the gradient loads first; everything below overlaps with them
    uint4 q[S::UNITS][8 / E::G];
    uint64_t kbits[S::UNITS];
#pragma unroll
    for (int u = 0; u < S::UNITS; ++u) {
        const int64_t i = t0 + (int64_t)(u * kThreads + tid) * 8;
        if (i < t1) {
#pragma unroll
            for (int h = 0; h < 8 / E::G; ++h) q[u][h] = ld_stream(row + (i + h * E::G) * E::BYTES);
            kbits[u] = MULTI ? load_idx8<IDXB == 0 ? 8 : IDXB>(p.idx, i) : 0;
        }
    }

    // scale of this tile: uniform if one segment covers it (the common case)
    __shared__ float sh_inv[UQ_MAX_SCALES];
    const int j0 = find_segment(p.seg_off, p.nseg, t0);
    const bool uniform = segment_end(p.seg_off, p.nseg, j0, p.d) >= t1;
    if (tid < p.scales.N) {
        const float inv = inv_scale(p.scales.s[tid], __ldg(p.W + j0));
        sh_inv[tid] = inv;
        if (uniform && (__float_as_uint(inv) & 0x7F800000u) == 0x7F800000u && p.status)
            atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
    }
    __syncthreads();
    const float inv_single = sh_inv[0];
    const PhiloxKey key = philox_key(p.seed);

#pragma unroll
    for (int u = 0; u < S::UNITS; ++u) {
        const int64_t i = t0 + (int64_t)(u * kThreads + tid) * 8;
        if (i >= t1) continue;
        float v[8];
#pragma unroll
        for (int h = 0; h < 8 / E::G; ++h) E::unpack(q[u][h], *(float(*)[E::G])(v + h * E::G));
        if (i + 8 > p.d) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (i + e >= p.d) v[e] = 0.0f;      // padding quantizes to level 0
        }

        // per-coordinate s_i / W_j
        float inv[8];
        if (uniform) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
                inv[e] = MULTI ? sh_inv[(kbits[u] >> (e * IDXB)) & ((1u << IDXB) - 1u) & (UQ_MAX_SCALES - 1)]
                               : inv_single;
        } else {
            int j = find_segment(p.seg_off, p.nseg, i);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                j = advance_segment(p.seg_off, p.nseg, j, i + e);
                const int k = MULTI ? (int)((kbits[u] >> (e * IDXB)) & ((1u << IDXB) - 1u)) : 0;
                inv[e] = inv_scale(p.scales.s[k & (UQ_MAX_SCALES - 1)], __ldg(p.W + j));
                if ((__float_as_uint(inv[e]) & 0x7F800000u) == 0x7F800000u && p.status)
                    atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
            }
        }

        // random words: coordinate c uses word c%4 of block c/4 (32-bit draws) or half
        // (c%8)%2 of word (c%8)/2 of block c/8 (16-bit draws)
        int z[8];
        if (RNG == 32) {
            const uint4 r0 = philox4x32_10(key, (uint64_t)(i >> 2), (uint32_t)m);
            const uint4 r1 = philox4x32_10(key, (uint64_t)(i >> 2) + 1, (uint32_t)m);
            const uint32_t w[8] = { r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w };
#pragma unroll
            for (int e = 0; e < 8; ++e)
                z[e] = apply_sign(v[e], level_draw23(scaled_magnitude(v[e], inv[e], p.cap), w[e]));
        } else {
            const uint4 r = philox4x32_10(key, (uint64_t)(i >> 3), (uint32_t)m);
            const uint32_t w[4] = { r.x, r.y, r.z, r.w };
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t h16 = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
                z[e] = apply_sign(v[e], level_draw16(scaled_magnitude(v[e], inv[e], p.cap), h16));
            }
        }

        if (FMT == UQ_FMT_I8) {
            uint2 out;
            out.x = (z[0] & 0xFF) | ((z[1] & 0xFF) << 8) | ((z[2] & 0xFF) << 16) | ((uint32_t)z[3] << 24);
            out.y = (z[4] & 0xFF) | ((z[5] & 0xFF) << 8) | ((z[6] & 0xFF) << 16) | ((uint32_t)z[7] << 24);
            st_stream((uint2 *)((char *)p.lev + (size_t)m * (size_t)p.stride + i), out);
        } else {
            uint32_t out = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) out |= (uint32_t)(z[e] & 0xF) << (4 * e);
            st_stream((uint32_t *)((char *)p.lev + (size_t)m * (size_t)(p.stride >> 1) + (i >> 1)), out);
        }
    }
}

template <int DT, int FMT, int RNG, int IDXB>
static cudaError_t launch(const EncodeParams &p, cudaStream_t st)
{
    using S = EncodeShape<DT>;
    const int64_t tiles = (p.d + S::TILE - 1) / S::TILE;
    const int64_t blocks = tiles * p.M;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    encode_kernel<DT, FMT, RNG, IDXB><<<(unsigned)blocks, kThreads, 0, st>>>(p);
    return cudaGetLastError();
}

template <int DT, int FMT, int RNG>
static cudaError_t dispatch_idx(const EncodeParams &p, int idx_bits, cudaStream_t st)
{
    switch (idx_bits) {
    case 0: return launch<DT, FMT, RNG, 0>(p, st);
    case 2: return launch<DT, FMT, RNG, 2>(p, st);
    case 4: return launch<DT, FMT, RNG, 4>(p, st);
    default: return launch<DT, FMT, RNG, 8>(p, st);
    }
}

template <int DT>
static cudaError_t dispatch_fmt(const EncodeParams &p, int fmt, int rng_bits, int idx_bits, cudaStream_t st)
{
    if (fmt == UQ_FMT_I8)
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I8, 32>(p, idx_bits, st)
                              : dispatch_idx<DT, UQ_FMT_I8, 16>(p, idx_bits, st);
    return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I4X2, 32>(p, idx_bits, st)
                          : dispatch_idx<DT, UQ_FMT_I4X2, 16>(p, idx_bits, st);
}

// idx_bits == 0 selects the single-scale quantizer (scales = {s}).
cudaError_t launch_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                          uint32_t *status, cudaStream_t st)
{
    EncodeParams p;
    p.g = g; p.lev = lev; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.seed = seed; p.nseg = L.nseg; p.M = L.M;
    p.cap = (float)scales.s[0];
    p.scales = scales;
    return L.dtype == UQ_F32 ? dispatch_fmt<UQ_F32>(p, fmt, rng_bits, idx_bits, st)
                             : dispatch_fmt<UQ_BF16>(p, fmt, rng_bits, idx_bits, st);
}

}  // namespace uq
