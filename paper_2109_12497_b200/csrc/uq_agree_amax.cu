// Agree-scale for the multi-scale quantizer with a by-product: while the M workers' gradients are
// read for the norms (Algorithm 2, line "MaxAllReduce Norm"), the per-coordinate maximum magnitude
// over the workers, amax_i = max_m |g^m_i|, is written out.  The shared scale index of a coordinate
// depends on the gradients only through amax_i (see uq_select.cu), so the selector can then run on
// the single row amax instead of on all M rows: one of the three passes that the multi-scale path
// makes over the gradients shrinks to a pass over 1/M of the bytes.
//
// A CTA owns one tile of kAmaxTile coordinates of ALL workers (the plain kernel: 8192 of one worker).
// A thread takes 8 consecutive coordinates per sub-tile of 2048; it walks the workers, eight at a
// time, adding each worker's squares (or magnitudes) to that worker's accumulator and folding the
// magnitudes into the 8 running maxima, which it stores after the last worker.  The per-worker
// accumulators are then reduced over the CTA in a fixed order and stored in scratch slots
// (tile + segment) laid out like the plain kernel's, for its own tile size, so the finalize kernel is shared.  The order of additions
// differs from the plain kernel's (another assignment of coordinates to threads), so the last bit
// of W may differ between the two; each is reproducible.
#include "uq_device.cuh"
#include "uq_norm.cuh"

namespace uq {

#ifndef UQ_AMAX_TILE
#define UQ_AMAX_TILE 8192
#endif
constexpr int kAmaxTile = UQ_AMAX_TILE;            // coordinates per CTA and per partial (swept: 2048 and 4096 are slower)
constexpr int kSub = kThreads * 8;                 // coordinates per sub-tile
constexpr int kSubs = kAmaxTile / kSub;            // sub-tiles per tile
constexpr int kChunk = 8;                          // workers whose accumulators a thread holds at once

// amax of 8 coordinates, kept in the element type's own magnitude bits:
// fp32: eight floats (|v|, combined with fmaxf like the selector does); bf16: four words of two
// 15-bit magnitudes (combined with the packed 16-bit maximum).
template <int DT> struct Amax8;
template <> struct Amax8<UQ_F32> {
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    __device__ __forceinline__ void load(const void *p)
    {
        const uint4 x = *(const uint4 *)p, y = *((const uint4 *)p + 1);
        a[0] = __uint_as_float(x.x); a[1] = __uint_as_float(x.y); a[2] = __uint_as_float(x.z); a[3] = __uint_as_float(x.w);
        a[4] = __uint_as_float(y.x); a[5] = __uint_as_float(y.y); a[6] = __uint_as_float(y.z); a[7] = __uint_as_float(y.w);
    }
    __device__ __forceinline__ void fold(const uint4 (&q)[2], const float (&v)[8])
    {
#pragma unroll
        for (int e = 0; e < 8; ++e) a[e] = fmaxf(a[e], fabsf(v[e]));
    }
    __device__ __forceinline__ void store(void *p) const
    {
        *(uint4 *)p = make_uint4(__float_as_uint(a[0]), __float_as_uint(a[1]), __float_as_uint(a[2]), __float_as_uint(a[3]));
        *((uint4 *)p + 1) = make_uint4(__float_as_uint(a[4]), __float_as_uint(a[5]), __float_as_uint(a[6]), __float_as_uint(a[7]));
    }
};
template <> struct Amax8<UQ_BF16> {
    uint32_t a[4] = {0u, 0u, 0u, 0u};
    __device__ __forceinline__ void load(const void *p)
    {
        const uint4 x = *(const uint4 *)p;
        a[0] = x.x; a[1] = x.y; a[2] = x.z; a[3] = x.w;
    }
    __device__ __forceinline__ void fold(const uint4 (&q)[1], const float (&)[8])
    {
        a[0] = __vmaxu2(a[0], q[0].x & 0x7FFF7FFFu);
        a[1] = __vmaxu2(a[1], q[0].y & 0x7FFF7FFFu);
        a[2] = __vmaxu2(a[2], q[0].z & 0x7FFF7FFFu);
        a[3] = __vmaxu2(a[3], q[0].w & 0x7FFF7FFFu);
    }
    __device__ __forceinline__ void store(void *p) const { *(uint4 *)p = make_uint4(a[0], a[1], a[2], a[3]); }
};

// Eight values per lane reduced over the warp together: three exchange rounds that halve the number
// of values a lane holds (a lane keeps the half selected by one of its lane bits and adds the
// partner's copy of that half), then two ordinary rounds on the single value left.  Nine 64-bit
// exchanges instead of forty; the order of additions is fixed.  Afterwards the lanes with
// (lane & 3) == 0 hold the warp totals: lane 4 * k' holds value number bitrev3(k')... the mapping is
// returned in `which` (the index 0..7 of the value this lane ends up with).
template <int NORM>
__device__ __forceinline__ double warp_reduce8(const double (&v)[8], int lane, int &which)
{
    double a[4], b[2], c;
    {
        const bool up = lane & 16;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const double send = up ? v[k] : v[4 + k];
            const double recv = __shfl_xor_sync(0xFFFFFFFFu, send, 16);
            a[k] = combine<NORM>(up ? v[4 + k] : v[k], recv);
        }
    }
    {
        const bool up = lane & 8;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const double send = up ? a[k] : a[2 + k];
            const double recv = __shfl_xor_sync(0xFFFFFFFFu, send, 8);
            b[k] = combine<NORM>(up ? a[2 + k] : a[k], recv);
        }
    }
    {
        const bool up = lane & 4;
        const double send = up ? b[0] : b[1];
        const double recv = __shfl_xor_sync(0xFFFFFFFFu, send, 4);
        c = combine<NORM>(up ? b[1] : b[0], recv);
    }
    c = combine<NORM>(c, __shfl_xor_sync(0xFFFFFFFFu, c, 2));
    c = combine<NORM>(c, __shfl_xor_sync(0xFFFFFFFFu, c, 1));
    which = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
    return c;
}

template <int DT, int NORM>
__global__ void __launch_bounds__(kThreads, 3)
norm_amax_kernel(const void *__restrict__ g, int64_t d, int64_t stride, int M, int nseg,
                 const int64_t *__restrict__ seg_off, int64_t ntiles, double *__restrict__ part, void *__restrict__ amax)
{
    grid_dependency_prologue();
    using E = Elem<DT>;
    constexpr int H = 8 / E::G;
    const int64_t tile = blockIdx.x;
    const int64_t t0 = tile * kAmaxTile;
    const int64_t t1 = min(t0 + (int64_t)kAmaxTile, d);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t slots = (size_t)(ntiles + nseg);
    const int j0 = warp_find_segment(seg_off, nseg, t0);

    const bool full = t1 - t0 == kAmaxTile;                         // else the ragged last tile
    if (segment_end(seg_off, nseg, j0, d) < t1) {
        // a tile that a segment boundary crosses (so there is a segment table): the norms worker by
        // worker through the shared out-of-line path, the maxima in a plain pass of their own
        for (int m = 0; m < M; ++m) {
            norm_mixed_tile<DT, NORM>((const char *)g + (size_t)m * (size_t)stride * E::BYTES, part + (size_t)m * slots, tile,
                                      t0, t1, d, nseg, seg_off);
            __syncthreads();                                        // its shared scratch is reused by the next worker
        }
        for (int s = 0; s < kSubs; ++s) {
            const int64_t i = t0 + (int64_t)s * kSub + tid * 8;
            if (i >= t1) break;                                     // the padded row makes a unit that starts before d readable
            Amax8<DT> am;
            for (int m = 0; m < M; ++m) {
                uint4 q[H];
                float v[8];
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    q[h] = ld_stream((const char *)g + ((size_t)m * (size_t)stride + (size_t)i + h * E::G) * E::BYTES);
                    E::unpack(q[h], *(float(*)[E::G])(v + h * E::G));
                }
                am.fold(q, v);
            }
            am.store((char *)amax + (size_t)i * E::BYTES);
        }
        return;
    }

    __shared__ double sh[kChunk][kWarps];
    for (int c0 = 0; c0 < M; c0 += kChunk) {
        Acc<NORM> acc[kChunk];
#pragma unroll 1
        for (int s = 0; s < kSubs; ++s) {
            const int64_t i = t0 + (int64_t)s * kSub + tid * 8;
            if (i >= t1) break;                                     // ragged tile: nothing of this sub-tile is mine
            const char *col = (const char *)g + (size_t)i * E::BYTES;
            Amax8<DT> am;
            if (c0 > 0) am.load((const char *)amax + (size_t)i * E::BYTES);   // the maxima of the workers before this chunk
            constexpr int B = DT == UQ_BF16 ? 8 : 4;                // workers whose loads are in flight together
#pragma unroll
            for (int k0 = 0; k0 < kChunk; k0 += B) {
                uint4 q[B][H];
#pragma unroll
                for (int k = 0; k < B; ++k) {
                    const int m = min(c0 + k0 + k, M - 1);          // beyond the last worker: a repeat that is not added
#pragma unroll
                    for (int h = 0; h < H; ++h) q[k][h] = ld_stream(col + ((size_t)m * (size_t)stride + h * E::G) * E::BYTES);
                }
#pragma unroll
                for (int k = 0; k < B; ++k) {
                    float v[8];
#pragma unroll
                    for (int h = 0; h < H; ++h) E::unpack(q[k][h], *(float(*)[E::G])(v + h * E::G));
                    if (c0 + k0 + k < M) {
                        if (full) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[k0 + k].add(v[e]);
                        } else {                                    // the row's padding beyond d is not data
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (i + e < t1) acc[k0 + k].add(v[e]);
                        }
                        am.fold(q[k], v);
                    }
                }
            }
            am.store((char *)amax + (size_t)i * E::BYTES);
        }
        // one partial per worker of the chunk, reduced over the CTA in a fixed order
        {
            static_assert(kChunk == 8, "warp_reduce8 takes eight values");
            double v[kChunk];
#pragma unroll
            for (int k = 0; k < kChunk; ++k) v[k] = acc[k].value();
            int which;
            const double w = warp_reduce8<NORM>(v, lane, which);
            if ((lane & 3) == 0) sh[which][warp] = w;
        }
        __syncthreads();
        if (tid < kChunk && c0 + tid < M) {
            double tot = sh[tid][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) tot = combine<NORM>(tot, sh[tid][w]);
            part[(size_t)(c0 + tid) * slots + tile + j0] = tot;
        }
        __syncthreads();
    }
}

// The finalize kernel of uq_agree.cu (same scratch layout).
cudaError_t launch_norm_finalize(const uq_layout &L, int norm, const double *part, int64_t ntiles, int tile_coords,
                                 float *W, uint32_t *status, cudaStream_t st);

int64_t norm_tiles_amax(int64_t d) { return (d + kAmaxTile - 1) / kAmaxTile; }

cudaError_t launch_agree_scale_amax(const uq_layout &L, const void *g, int norm, float *W, void *amax, uint32_t *status,
                                    void *workspace, cudaStream_t st)
{
    const int64_t ntiles = norm_tiles_amax(L.d);
    double *part = (double *)workspace;
    if (L.d > 0) {
        if (ntiles > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
        const unsigned nb = (unsigned)ntiles;
        if (L.dtype == UQ_F32) {
            if (norm == UQ_NORM_L2) launch_k(norm_amax_kernel<UQ_F32, UQ_NORM_L2>, nb, kThreads, st, g, L.d, L.worker_stride, L.M, L.nseg, L.seg_off, ntiles, part, amax);
            else launch_k(norm_amax_kernel<UQ_F32, UQ_NORM_LINF>, nb, kThreads, st, g, L.d, L.worker_stride, L.M, L.nseg, L.seg_off, ntiles, part, amax);
        } else {
            if (norm == UQ_NORM_L2) launch_k(norm_amax_kernel<UQ_BF16, UQ_NORM_L2>, nb, kThreads, st, g, L.d, L.worker_stride, L.M, L.nseg, L.seg_off, ntiles, part, amax);
            else launch_k(norm_amax_kernel<UQ_BF16, UQ_NORM_LINF>, nb, kThreads, st, g, L.d, L.worker_stride, L.M, L.nseg, L.seg_off, ntiles, part, amax);
        }
    }
    return launch_norm_finalize(L, norm, part, ntiles, kAmaxTile, W, status, st);
}

}  // namespace uq
