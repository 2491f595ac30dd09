// Pieces of the norm reduction shared by the two agree-scale kernels: the accumulators of the two
// norms, the fixed-order warp reduction, and the out-of-line path for a tile that several segments
// cross.
#pragma once
#include "uq_device.cuh"

namespace uq {

template <int NORM> struct Acc;
template <> struct Acc<UQ_NORM_L2> {            // sum of exact binary64 squares
    double a = 0.0;
    // x*x is exact in binary64, so the fused multiply-add rounds once, exactly like add(a, x*x)
    __device__ __forceinline__ void add(float v) { double x = (double)v; a = __fma_rn(x, x, a); }
    __device__ __forceinline__ void merge(double o) { a = __dadd_rn(a, o); }
    __device__ __forceinline__ double value() const { return a; }
};
template <> struct Acc<UQ_NORM_LINF> {          // max of |v| as an integer compare of the bits
    uint32_t a = 0u;                            // (NaN > Inf > finite, so non-finite input survives)
    __device__ __forceinline__ void add(float v) { a = max(a, __float_as_uint(v) & 0x7FFFFFFFu); }
    __device__ __forceinline__ void merge(double o) { a = max(a, (uint32_t)o); }
    __device__ __forceinline__ double value() const { return (double)a; }
};

template <int NORM> __device__ __forceinline__ double combine(double x, double y)
{
    return NORM == UQ_NORM_L2 ? __dadd_rn(x, y) : fmax(x, y);
}

template <int NORM> __device__ __forceinline__ double warp_reduce(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = combine<NORM>(x, __shfl_xor_sync(0xFFFFFFFFu, x, o));
    return x;
}

// A tile crossed by several segments (kept out of line: it is rare and must not cost the common
// path registers).  Warp w owns the chunk of kNormTile / kWarps consecutive coordinates and walks
// the pieces of segments inside it (lane-strided scalar loads, one warp reduction per piece).  A
// segment that lies inside one chunk has a single writer and goes straight to its slot; a piece
// that touches a chunk border may continue in the neighbouring chunk, so those are parked in
// shared memory and thread 0 adds them up in chunk order: the order of additions depends only on
// (d, seg_off).
template <int DT, int NORM>
__device__ __noinline__ void norm_mixed_tile(const char *__restrict__ row, double *__restrict__ prow, int64_t tile,
                                             int64_t t0, int64_t t1, int64_t d, int nseg,
                                             const int64_t *__restrict__ seg_off)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int CHUNK = kNormTile / kWarps;
    __shared__ double sh_head[kWarps], sh_tail[kWarps];
    __shared__ int sh_head_seg[kWarps], sh_tail_seg[kWarps];     // -1: no such piece
    __shared__ int sh_head_open[kWarps];                          // head piece reaches the chunk's end
    const int64_t c0 = t0 + (int64_t)warp * CHUNK;
    const int64_t c1 = min(c0 + CHUNK, t1);
    int head_seg = -1, tail_seg = -1, head_open = 0;
    double head = 0.0, tail = 0.0;
    if (c0 < c1) {
        int j = warp_find_segment(seg_off, nseg, c0);
        int64_t a = c0;
        while (a < c1) {
            const int64_t seg_a = __ldg(seg_off + j);
            const int64_t seg_b = j + 1 < nseg ? __ldg(seg_off + j + 1) : d;   // clamp a bad table
            const int64_t b = min(max(seg_b, a), c1);
            if (b > a) {
                Acc<NORM> acc;
                for (int64_t i = a + lane; i < b; i += 32) {
                    float v = DT == UQ_F32 ? __ldg((const float *)row + i)
                                           : __uint_as_float((uint32_t)__ldg((const uint16_t *)row + i) << 16);
                    acc.add(v);
                }
                const double w = warp_reduce<NORM>(acc.value());
                const bool from_before = a == c0 && seg_a < c0;      // may continue from the left chunk
                const bool goes_on = b == c1 && seg_b > c1;          // may continue in the right chunk
                if (from_before) { head = w; head_seg = j; head_open = goes_on; }
                else if (goes_on) { tail = w; tail_seg = j; }
                else if (lane == 0) prow[tile + j] = w;
            }
            a = b;
            if (a < c1) { if (j + 1 < nseg) ++j; else break; }
        }
    }
    if (lane == 0) {
        sh_head[warp] = head; sh_tail[warp] = tail;
        sh_head_seg[warp] = head_seg; sh_tail_seg[warp] = tail_seg; sh_head_open[warp] = head_open;
    }
    __syncthreads();
    if (tid == 0) {
        int cur = -1;                  // segment whose pieces are being added up
        double sum = 0.0;
        for (int w = 0; w < kWarps; ++w) {
            if (sh_head_seg[w] >= 0) {
                if (cur == sh_head_seg[w]) sum = combine<NORM>(sum, sh_head[w]);
                else { if (cur >= 0) prow[tile + cur] = sum; cur = sh_head_seg[w]; sum = sh_head[w]; }
                if (!sh_head_open[w]) { prow[tile + cur] = sum; cur = -1; }
            }
            if (sh_tail_seg[w] >= 0) {
                if (cur >= 0) prow[tile + cur] = sum;
                cur = sh_tail_seg[w]; sum = sh_tail[w];
            }
        }
        if (cur >= 0) prow[tile + cur] = sum;
    }
}

}  // namespace uq
