// GlobalRandKMaxNorm / GlobalRandKMaxNormMultiScale (Sections "GlobalRandKMaxNorm Compression" and
// "GlobalRandKMaxNormMultiScale Compression"): all workers keep the same K coordinates, chosen
// uniformly from a shared seed, and the quantizer of Algorithm 1 / 2 runs on the K-vector.
//
// This file holds what the sparsifier adds around the dense path: the choice of the coordinates
// fused with the gather into a compact [M][K] buffer, and the scatter of the reconstructed values
// (into a dense vector, or straight into the parameters).  K is small (10^4 in the paper's
// experiments), so these kernels are latency-bound: one thread per chosen coordinate, all M loads
// of a thread in flight together.
#include "uq_device.cuh"

namespace uq {

// The chosen coordinates are the first K images of a keyed permutation of [0, d): an alternating
// Feistel network on b = max(2, ceil(log2 d)) bits (left part b/2 bits, right part the rest, the
// parts swap every round) with a Philox word as round function, restricted to [0, d) by cycle
// walking.  8 rounds; 24 when b < 8, where the round functions are only one to three bits wide.
__device__ __forceinline__ uint64_t randk_network(uint64_t x, int b, const PhiloxKey &key)
{
    int a = b >> 1, c = b - a;
    uint64_t L = x >> c, R = x & ((1ull << c) - 1ull);
    const uint32_t rounds = b < 8 ? 24u : 8u;
    for (uint32_t r = 0; r < rounds; ++r) {
        const uint4 w = philox4x32_10(key, (uint32_t)R, r, 0u, 0x4B646E52u);
        const uint64_t nr = L ^ ((uint64_t)w.x & ((1ull << a) - 1ull));
        L = R; R = nr;
        const int t = a; a = c; c = t;
    }
    return (L << c) | R;
}

constexpr int kWalkLimit = 256;      // a walk this long has probability below 2^-256

struct RandkParams {
    const void *g;
    void *gk;
    int64_t *sel;
    uint32_t *status;
    int64_t d, stride, K, gk_stride;
    int32_t M, bits;
    PhiloxKey key;
};

template <int DT>
__global__ void __launch_bounds__(kThreads) randk_gather_kernel(const __grid_constant__ RandkParams p)
{
    grid_dependency_prologue();
    using T = typename std::conditional<DT == UQ_F32, uint32_t, uint16_t>::type;
    const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (t >= p.gk_stride) return;
    T *dst = (T *)p.gk + t;
    if (t >= p.K) {                                              // row padding
        for (int m = 0; m < p.M; ++m) dst[(size_t)m * (size_t)p.gk_stride] = 0;
        return;
    }
    uint64_t x = (uint64_t)t;
    int step = 0;
    do x = randk_network(x, p.bits, p.key); while (x >= (uint64_t)p.d && ++step < kWalkLimit);
    if (x >= (uint64_t)p.d) {                                    // never expected; stay in range
        x = (uint64_t)t;
        if (p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_BAD_INDEX);
    }
    p.sel[t] = (int64_t)x;
    const T *src = (const T *)p.g + x;
    int m = 0;
    for (; m + 8 <= p.M; m += 8) {                               // eight workers' loads in flight
        T v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldg(src + (size_t)(m + k) * (size_t)p.stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) dst[(size_t)(m + k) * (size_t)p.gk_stride] = v[k];
    }
    for (; m < p.M; ++m) dst[(size_t)m * (size_t)p.gk_stride] = __ldg(src + (size_t)m * (size_t)p.stride);
}

// out[sel[t]] = vals[t] (vals == NULL: 0), or theta[sel[t]] -= lr * vals[t] when UPDATE.
template <bool UPDATE>
__global__ void __launch_bounds__(kThreads) randk_scatter_kernel(int64_t d, int64_t K, const int64_t *sel,
                                                                 const float *vals, float *dst, float lr,
                                                                 uint32_t *status)
{
    grid_dependency_prologue();
    const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (t >= K) return;
    const int64_t i = __ldg(sel + t);
    if (i < 0 || i >= d) {
        if (status) atomicOr(status, (uint32_t)UQ_STATUS_BAD_INDEX);
        return;
    }
    const float v = vals ? __ldg(vals + t) : 0.0f;
    if (UPDATE) dst[i] = __fsub_rn(dst[i], __fmul_rn(lr, v));    // Algorithm 1 / 2, line "Update parameters"
    else dst[i] = v;
}

cudaError_t launch_randk_gather(const uq_layout &L, const void *g, int64_t K, uint64_t seed, int64_t *sel,
                                void *gk, int64_t gk_stride, uint32_t *status, cudaStream_t st)
{
    if (gk_stride == 0) return cudaSuccess;
    RandkParams p;
    p.g = g; p.gk = gk; p.sel = sel; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.K = K; p.gk_stride = gk_stride; p.M = L.M;
    p.bits = 2;
    while (((int64_t)1 << p.bits) < L.d) ++p.bits;
    p.key = philox_key(seed);
    const int64_t blocks = (gk_stride + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (L.dtype == UQ_F32) launch_k(randk_gather_kernel<UQ_F32>, (unsigned)blocks, kThreads, st, p);
    else launch_k(randk_gather_kernel<UQ_BF16>, (unsigned)blocks, kThreads, st, p);
    return cudaGetLastError();
}

cudaError_t launch_randk_scatter(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *dst, bool update,
                                 float lr, uint32_t *status, cudaStream_t st)
{
    if (K == 0) return cudaSuccess;
    const int64_t blocks = (K + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (update) launch_k(randk_scatter_kernel<true>, (unsigned)blocks, kThreads, st, d, K, sel, vals, dst, lr, status);
    else launch_k(randk_scatter_kernel<false>, (unsigned)blocks, kThreads, st, d, K, sel, vals, dst, lr, status);
    return cudaGetLastError();
}

}  // namespace uq
