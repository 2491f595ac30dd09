// Host side of the encoders: fills the kernel parameters and picks the translation unit that holds
// the kernels of the element type and draw width (uq_encode.cuh has the kernels).
#include "uq_encode.cuh"

namespace uq {

// idx_bits == 0 selects the single-scale quantizer (scales = {s}).
cudaError_t launch_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                          uint32_t *status, cudaStream_t st)
{
    EncodeParams p;
    p.g = g; p.lev = lev; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M; p.worker0 = L.worker0; p.coord0 = L.coord0;
    p.key = philox_key(seed);
    // CTA order (set in the kernel): the tiles are walked back to front.  The kernel before this one
    // in a step (agree-scale or the selector) ends on the high tiles, so part of what is read first
    // is still in L2, and the kernel ends on the lowest tiles, where the aggregation starts.
    p.cap = (float)scales.s[0];
    p.scales = scales;
    if (L.dtype == UQ_F32)
        return rng_bits == 32 ? launch_encode_f32_r32(p, fmt, idx_bits, st) : launch_encode_f32_r16(p, fmt, idx_bits, st);
    return rng_bits == 32 ? launch_encode_bf16_r32(p, fmt, idx_bits, st) : launch_encode_bf16_r16(p, fmt, idx_bits, st);
}

}  // namespace uq
