// Host side of the encoders: fills the kernel parameters and picks the translation unit that holds
// the kernels of the element type and draw width (uq_encode.cuh has the kernels).
#include "uq_encode.cuh"

namespace uq {

cudaError_t launch_select(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          int idx_bits, uint8_t *idx, uint32_t *status, cudaStream_t st);

static cudaError_t launch_encode_any(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                                     uint8_t *idx, int idx_bits, bool select, uint64_t seed, int rng_bits, int fmt,
                                     void *lev, uint32_t *status, cudaStream_t st, float *out = nullptr)
{
    EncodeParams p;
    p.out = out;
    p.v.g = g; p.v.W = W; p.v.seg_off = L.seg_off; p.v.d = L.d; p.v.stride = L.worker_stride; p.v.nseg = L.nseg; p.v.M = L.M;
    p.v.s_hat = (float)scales.s[0];
    p.v.scales = scales;
    p.lev = lev; p.idx = idx; p.status = status; p.select = select ? 1 : 0;
    p.worker0 = L.worker0; p.coord0 = L.coord0;
    p.key = philox_key(seed);
    // CTA order (set in the kernel): the tiles are walked back to front.  The kernel before this one
    // in a step (agree-scale or the selector) ends on the high tiles, so part of what is read first
    // is still in L2, and the kernel ends on the lowest tiles, where the aggregation starts.
    if (L.dtype == UQ_F32)
        return rng_bits == 32 ? launch_encode_f32_r32(p, fmt, idx_bits, st) : launch_encode_f32_r16(p, fmt, idx_bits, st);
    return rng_bits == 32 ? launch_encode_bf16_r32(p, fmt, idx_bits, st) : launch_encode_bf16_r16(p, fmt, idx_bits, st);
}

// idx_bits == 0 selects the single-scale quantizer (scales = {s}).
cudaError_t launch_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                          uint32_t *status, cudaStream_t st)
{
    return launch_encode_any(L, g, W, scales, const_cast<uint8_t *>(idx), idx_bits, false, seed, rng_bits, fmt, lev, status, st);
}

// Quantization, sum over the workers and reconstruction in one kernel (decode mode of the encoder):
// int8 levels and at most kWorkerGroup workers, so that the CTA of a tile sees every worker's levels,
// and 16-bit draws (with 32-bit draws the one kernel is no faster than the two: measured).
bool encode_decode_fused(const uq_layout &L, int fmt, int rng_bits)
{
    return fmt == UQ_FMT_I8 && L.M <= kWorkerGroup && rng_bits == 16;
}

cudaError_t launch_encode_decode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                                 const uint8_t *idx, int idx_bits, uint64_t seed, void *lev, float *out, uint32_t *status,
                                 cudaStream_t st)
{
    return launch_encode_any(L, g, W, scales, const_cast<uint8_t *>(idx), idx_bits, false, seed, 16, UQ_FMT_I8, lev, status, st, out);
}

// Scale selection, scale sharing and quantization in one kernel: a CTA that takes a tile through
// all workers reads their rows once more first (max over the workers of every magnitude), finds
// and stores the shared indices, and quantizes with them; the second read of the rows comes from
// L2.  With more workers than one CTA takes (M > kWorkerGroup) the selector runs as a kernel of
// its own in front.  idx and lev are bit for bit those of the two separate calls either way.
cudaError_t launch_select_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales, int idx_bits,
                                 uint64_t seed, int rng_bits, int fmt, uint8_t *idx, void *lev, uint32_t *status,
                                 cudaStream_t st)
{
    if (L.M > kWorkerGroup) {
        const cudaError_t e = launch_select(L, g, W, scales, idx_bits, idx, status, st);
        if (e != cudaSuccess) return e;
        return launch_encode_any(L, g, W, scales, idx, idx_bits, false, seed, rng_bits, fmt, lev, status, st);
    }
    return launch_encode_any(L, g, W, scales, idx, idx_bits, true, seed, rng_bits, fmt, lev, status, st);
}

// Select mode and decode mode of the encoder together: everything of a multi-scale step behind the
// scale agreement in one kernel.  The caller has checked encode_decode_fused().
cudaError_t launch_select_encode_decode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                                        int idx_bits, uint64_t seed, uint8_t *idx, void *lev, float *out, uint32_t *status,
                                        cudaStream_t st)
{
    return launch_encode_any(L, g, W, scales, idx, idx_bits, true, seed, 16, UQ_FMT_I8, lev, status, st, out);
}

}  // namespace uq
