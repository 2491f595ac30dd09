// The encoder's kernels for bf16 gradients and 16-bit draws (see uq_encode.cuh).
#include "uq_encode.cuh"

namespace uq {

cudaError_t launch_encode_bf16_r16(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st)
{
    return dispatch_fmt<UQ_BF16, 16>(p, fmt, idx_bits, st);
}

}  // namespace uq
