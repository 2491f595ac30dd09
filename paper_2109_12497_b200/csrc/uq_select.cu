// Per-coordinate scale index with scale sharing
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
#include "uq_device.cuh"

namespace uq {

struct SelectParams {
    const void *g;
    uint8_t *idx;
    const float *W;
    const int64_t *seg_off;
    uint32_t *status;
    int64_t d, stride;
    int32_t nseg, M;
    float s_hat;
    ScaleSet scales;
};

constexpr int kSelectTile = kThreads * 8;

__device__ __forceinline__ float inv_scale_sel(int32_t s, float W)
{
    return W > 0.0f ? __fdiv_rn((float)s, W) : 0.0f;
}

template <int DT, int IDXB>
__global__ void __launch_bounds__(kThreads) select_kernel(const SelectParams p)
{
    using E = Elem<DT>;
    const int64_t t0 = (int64_t)blockIdx.x * kSelectTile;
    const int64_t t1 = min(t0 + (int64_t)kSelectTile, p.d);
    const int tid = threadIdx.x;
    const int64_t i = t0 + (int64_t)tid * 8;
    const int N = p.scales.N;

    float amax[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) amax[e] = 0.0f;
    if (i < t1) {
        const char *col = (const char *)p.g + (size_t)i * E::BYTES;
        int m = 0;
        // four workers' loads in flight at a time
        for (; m + 4 <= p.M; m += 4) {
            uint4 q[4][8 / E::G];
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int h = 0; h < 8 / E::G; ++h)
                    q[k][h] = ld_stream(col + ((size_t)(m + k) * (size_t)p.stride + h * E::G) * E::BYTES);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float v[8];
#pragma unroll
                for (int h = 0; h < 8 / E::G; ++h) E::unpack(q[k][h], *(float(*)[E::G])(v + h * E::G));
#pragma unroll
                for (int e = 0; e < 8; ++e) amax[e] = fmaxf(amax[e], fabsf(v[e]));
            }
        }
        for (; m < p.M; ++m) {
            float v[8];
#pragma unroll
            for (int h = 0; h < 8 / E::G; ++h) {
                uint4 q = ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES);
                E::unpack(q, *(float(*)[E::G])(v + h * E::G));
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) amax[e] = fmaxf(amax[e], fabsf(v[e]));
        }
    }

    __shared__ float sh_inv[UQ_MAX_SCALES];
    const int j0 = find_segment(p.seg_off, p.nseg, t0);
    const bool uniform = segment_end(p.seg_off, p.nseg, j0, p.d) >= t1;
    if (tid < N) sh_inv[tid] = inv_scale_sel(p.scales.s[tid], __ldg(p.W + j0));
    __syncthreads();
    if (i >= t1) return;

    uint64_t packed = 0;
    int j = uniform ? j0 : find_segment(p.seg_off, p.nseg, i);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int k = 0;
        if (i + e < p.d) {                          // padding keeps index 0
            if (uniform) {
                for (int kk = 1; kk < N; ++kk)
                    if (__fmul_rn(amax[e], sh_inv[kk]) <= p.s_hat) k = kk;
            } else {
                j = advance_segment(p.seg_off, p.nseg, j, i + e);
                const float Wj = __ldg(p.W + j);
                for (int kk = 1; kk < N; ++kk)
                    if (__fmul_rn(amax[e], inv_scale_sel(p.scales.s[kk], Wj)) <= p.s_hat) k = kk;
            }
        }
        packed |= (uint64_t)k << (e * IDXB);
    }
    if (IDXB == 2) *(uint16_t *)(p.idx + (i >> 2)) = (uint16_t)packed;
    else if (IDXB == 4) *(uint32_t *)(p.idx + (i >> 1)) = (uint32_t)packed;
    else *(uint64_t *)(p.idx + i) = packed;
}

template <int DT>
static cudaError_t dispatch(const SelectParams &p, int idx_bits, cudaStream_t st)
{
    const int64_t blocks = (p.d + kSelectTile - 1) / kSelectTile;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (idx_bits == 2) select_kernel<DT, 2><<<(unsigned)blocks, kThreads, 0, st>>>(p);
    else if (idx_bits == 4) select_kernel<DT, 4><<<(unsigned)blocks, kThreads, 0, st>>>(p);
    else select_kernel<DT, 8><<<(unsigned)blocks, kThreads, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_select(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          int idx_bits, uint8_t *idx, uint32_t *status, cudaStream_t st)
{
    SelectParams p;
    p.g = g; p.idx = idx; p.W = W; p.seg_off = L.seg_off; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M;
    p.s_hat = (float)scales.s[0];
    p.scales = scales;
    return L.dtype == UQ_F32 ? dispatch<UQ_F32>(p, idx_bits, st) : dispatch<UQ_BF16>(p, idx_bits, st);
}

}  // namespace uq
