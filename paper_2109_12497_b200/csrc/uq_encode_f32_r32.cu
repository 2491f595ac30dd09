// The encoder's kernels for binary32 gradients and 32-bit draws (see uq_encode.cuh).
#include "uq_encode.cuh"

namespace uq {

cudaError_t launch_encode_f32_r32(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st)
{
    return dispatch_fmt<UQ_F32, 32>(p, fmt, idx_bits, st);
}

}  // namespace uq
