// Per-coordinate scale index with scale sharing: the pieces shared by the selector's kernels and
// by the encoder that selects for itself
// (Section "QSGDMaxNormMultiScale Quantization": the inequality defining s*_i and the
//  "scale sharing" rule s*_i = min_m s*^{,m}_i; Algorithm 2 lines "Compute coordinate scales"
//  and "Scale sharing").
//
// Worker m's own index is k^m_i = max{k : |g^m_i| * inv_k <= s_hat} with inv_k = s_k / W_j
// non-decreasing in k.  Multiplication by a positive constant is monotone in binary32, so each
// test "|v| * inv_k <= s_hat" can only switch from true to false as |v| grows: k^m_i is
// non-increasing in |g^m_i|, and min_m k^m_i = k(max_m |g^m_i|) exactly.  The kernel therefore
// folds the min-all-reduce into a max over the M resident buffers followed by one threshold
// search per coordinate; the result is bit-identical to selecting per worker and taking the min.
#pragma once
#include "uq_device.cuh"

namespace uq {

// What the selection reads.
struct SelectView {
    const void *g;
    const float *W;
    const int64_t *seg_off;
    int64_t d, stride;
    int32_t nseg, M;
    float s_hat;
    ScaleSet scales;
};

__device__ __forceinline__ float inv_scale_sel(int32_t s, float W)
{
    return W > 0.0f ? __fdiv_rn((float)s, W) : 0.0f;
}

// The general path for one thread's 8 coordinates (row crossed by a segment boundary): the test
// is evaluated as written, with one division per scale and coordinate.  Rare, kept out of line.
static __device__ __noinline__ uint64_t select_general(const SelectView &p, int64_t i, const uint32_t (&amag)[8], int idxb,
                                                 int j)      // j: a segment at or before coordinate i's
{
    uint64_t packed = 0;
    for (int e = 0; e < 8; ++e) {
        int k = 0;
        if (i + e < p.d) {                                          // padding keeps index 0
            j = advance_segment(p.seg_off, p.nseg, j, i + e);
            const float Wj = __ldg(p.W + j), a = __uint_as_float(amag[e]);
            for (int kk = 1; kk < p.scales.N; ++kk)
                if (__fmul_rn(a, inv_scale_sel(p.scales.s[kk], Wj)) <= p.s_hat) k = kk;
        }
        packed |= (uint64_t)k << (e * idxb);
    }
    return packed;
}

// max over the workers of the magnitude bits of coordinates i .. i + 7 (as binary32 patterns)
template <int DT>
__device__ __forceinline__ void unit_max_magnitude(const SelectView &p, int64_t i, bool active, uint32_t (&amag)[8])
{
    using E = Elem<DT>;
    constexpr int H = 8 / E::G;
    if (DT == UQ_F32) {
        float amax[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) amax[e] = 0.0f;
        if (active) {
            const char *col = (const char *)p.g + (size_t)i * E::BYTES;
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
        // bf16 magnitudes order like unsigned 15-bit integers: packed 16-bit max, no unpacking
        uint32_t am[4] = {0u, 0u, 0u, 0u};
        if (active) {
            const char *col = (const char *)p.g + (size_t)i * E::BYTES;
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
}

// The packed shared indices of the 8 coordinates starting at i (the calling thread's unit; the
// warp's units form the row of 256 coordinates starting at row0 < d).  Every warp looks up the
// segment of its own row and builds the threshold table of that segment in its own slice `thr`
// of shared memory (2 * UQ_MAX_SCALES words): entry k is the largest magnitude that passes scale
// k, -1 beyond the last scale.  LEVELS >= ceil(log2 N): the search is a bisection over the table.
// Must be called by whole warps.
template <int DT, int IDXB, int LEVELS>
__device__ __forceinline__ uint64_t select_unit(const SelectView &p, int64_t i, int64_t row0, int32_t *thr_table)
{
    const int lane = threadIdx.x & 31;
    const bool active = i < p.d;
    uint32_t amag[8];
    unit_max_magnitude<DT>(p, i, active, amag);
    const int64_t row1 = min(row0 + 256, p.d);
    const int j0 = warp_find_segment(p.seg_off, p.nseg, row0);
    uint64_t packed = 0;
    if (segment_end(p.seg_off, p.nseg, j0, p.d) >= row1) {
        int32_t thr = -1;
        if (lane < p.scales.N) thr = pass_threshold(inv_scale_sel(p.scales.s[lane], __ldg(p.W + j0)), p.s_hat);
        __syncwarp();
        thr_table[lane] = thr;
        __syncwarp();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int32_t a = (int32_t)amag[e];
            int k = 0;
#pragma unroll
            for (int step = 1 << (LEVELS - 1); step >= 1; step >>= 1)
                if (a <= thr_table[k + step]) k += step;            // k + step < 2^LEVELS <= 16
            if (i + e >= p.d) k = 0;                                // padding keeps index 0
            packed |= (uint64_t)k << (e * IDXB);
        }
    } else if (active) {
        packed = select_general(p, i, amag, IDXB, j0);
    }
    return packed;
}

// Stores the packed indices of the unit that starts at coordinate i.
template <int IDXB> __device__ __forceinline__ void store_unit_indices(uint8_t *idx, int64_t i, uint64_t packed)
{
    if (IDXB == 1) idx[i >> 3] = (uint8_t)packed;
    else if (IDXB == 2) *(uint16_t *)(idx + (i >> 2)) = (uint16_t)packed;
    else if (IDXB == 4) *(uint32_t *)(idx + (i >> 1)) = (uint32_t)packed;
    else *(uint64_t *)(idx + i) = packed;
}

}  // namespace uq
