// One whole multi-scale step in ONE kernel for small gradients (Algorithm 2, lines "MaxAllReduce
// Norm" to "Reconstruct gradient"; one segment, at most 8 workers): the cooperative-grid form of
// uq_small.cu with scale selection and scale sharing added to its second pass.
//
// After the scale agreement (uq_small.cuh) a thread owns 8 coordinates of ALL workers, as in the
// fused selector + encoder (uq_select_encode.cu): it forms max_m |g^m_i| (the shared index is a
// function of that maximum), finds the 8 shared indices by bisection over the exact pass
// thresholds, stores them, and then quantizes every worker's unit with the factors s_k / W of its
// coordinates, adds the levels in 16-bit lanes and writes W * sum / (s_k * M).  Indices, levels,
// sums and the reconstruction are bit for bit those of the separate calls given the same W.
// The level format is a run-time switch here (the kernel is latency-bound; the template
// parameters that remain are the element type, the norm, the draw width and the index width).
#include "uq_small.cuh"

namespace uq {

__device__ __forceinline__ void store_unit_any(int fmt, uint32_t lo, uint32_t hi, char *row, int64_t i)
{
    if (fmt == UQ_FMT_I8) store_unit<UQ_FMT_I8>(lo, hi, row + i, nullptr);
    else if (fmt == UQ_FMT_I4X2) store_unit<UQ_FMT_I4X2>(lo, hi, row + (i >> 1), nullptr);
    else store_unit<UQ_FMT_I2X4>(lo, hi, row + (i >> 2), nullptr);
}

template <int DT, int NORM, int RNG, int IDXB>
__global__ void __launch_bounds__(kThreads, 2) small_step_multi_kernel(const __grid_constant__ SmallParams p)
{
    using E = Elem<DT>;
    constexpr int H = 8 / E::G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t nunits = (p.d + 7) >> 3;
    const int64_t ustep = (int64_t)gridDim.x * kThreads;
    float W;
    if (!small_agree<DT, NORM>(p, W)) return;

    // lane k of every warp holds the factor s_k / W, the reconstruction factor W / (s_k * M) and the
    // pass threshold of scale k (one segment: the same for the whole vector)
    __shared__ int32_t sh_thr[kWarps][32];
    const float cap = (float)p.scales.s[0];
    const int32_t s_lane = p.scales.s[lane & (UQ_MAX_SCALES - 1)];
    const float inv_lane = inv_scale(s_lane, W);
    const float c_lane = __fdiv_rn(W, __fmul_rn((float)s_lane, (float)p.M));
    sh_thr[warp][lane] = lane < p.scales.N ? pass_threshold(inv_lane, cap) : -1;
    __syncwarp();
    if (blockIdx.x == 0 && warp == 0) {
        const bool overflow = lane < p.scales.N && not_finite(inv_lane);
        if (__any_sync(0xFFFFFFFFu, overflow) && lane == 0 && p.status)
            atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
    }
    const int32_t *T = sh_thr[warp];
    int top = 1;
    while (2 * top < p.scales.N) top *= 2;                          // the bisection's first step
    const size_t row_bytes = (size_t)(p.stride >> p.fmt);
    constexpr int G = 2;                                            // workers whose loads are in flight together

    // the loop bound is the same for all lanes of a warp (the shuffles below need every lane)
    for (int64_t ub = (int64_t)blockIdx.x * kThreads + (tid & ~31); ub < nunits; ub += ustep) {
        const int64_t u = ub + lane;
        const bool active = u < nunits;
        const int64_t i = u << 3;
        const char *col = (const char *)p.g + (size_t)i * E::BYTES;

        // max over the workers of the magnitude bits
        uint32_t amag[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) amag[e] = 0u;
        if (active) {
            for (int m = 0; m < p.M; ++m) {
                uint4 q[H];
#pragma unroll
                for (int h = 0; h < H; ++h) q[h] = ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES);
                if (DT == UQ_F32) {
                    const uint32_t w[8] = { q[0].x, q[0].y, q[0].z, q[0].w, q[H - 1].x, q[H - 1].y, q[H - 1].z, q[H - 1].w };
#pragma unroll
                    for (int e = 0; e < 8; ++e) amag[e] = max(amag[e], w[e] & 0x7FFFFFFFu);
                } else {
                    const uint32_t w[4] = { q[0].x, q[0].y, q[0].z, q[0].w };
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        amag[2 * k] = max(amag[2 * k], (w[k] << 16) & 0x7FFFFFFFu);
                        amag[2 * k + 1] = max(amag[2 * k + 1], w[k] & 0x7FFF0000u);
                    }
                }
            }
        }

        // the shared indices of my 8 coordinates, their factors and reconstruction factors
        uint64_t packed = 0;
        float inv[8], c[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int32_t a = (int32_t)amag[e];
            int k = 0;
            for (int step = top; step >= 1; step >>= 1)
                if (a <= T[k + step]) k += step;                    // k + step < 2 * top <= 16 + 15
            if (!active || i + e >= p.d) k = 0;                     // padding keeps index 0
            packed |= (uint64_t)k << (e * IDXB);
            inv[e] = __shfl_sync(0xFFFFFFFFu, inv_lane, k);
            c[e] = __shfl_sync(0xFFFFFFFFu, c_lane, k);
        }
        if (!active) continue;                                      // no warp-wide operation below
        if (IDXB == 1) p.idx[i >> 3] = (uint8_t)packed;
        else if (IDXB == 2) *(uint16_t *)(p.idx + (i >> 2)) = (uint16_t)packed;
        else if (IDXB == 4) *(uint32_t *)(p.idx + (i >> 1)) = (uint32_t)packed;
        else *(uint64_t *)(p.idx + i) = packed;

        // every worker's unit again (from L2), quantized with the shared factors, levels added
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        const uint32_t blk_lo = (uint32_t)blk, blk_hi = (uint32_t)(blk >> 32);
        const bool ragged = i + 8 > p.d;
        uint32_t even[2] = {0u, 0u}, odd[2] = {0u, 0u};             // level sums, biased by 128, in 16-bit lanes
        for (int m0 = 0; m0 < p.M; m0 += G) {
            uint4 q[G][H];
#pragma unroll
            for (int n = 0; n < G; ++n) {
                const int m = min(m0 + n, p.M - 1);                 // beyond the last worker: a harmless repeat
#pragma unroll
                for (int h = 0; h < H; ++h) q[n][h] = ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES);
            }
#pragma unroll
            for (int n = 0; n < G; ++n) {
                const UnitWords<RNG> rw = unit_words<RNG>(p.key, blk_lo, blk_hi, (uint32_t)(m0 + n + p.worker0));
                float v[8];
#pragma unroll
                for (int h = 0; h < H; ++h) E::unpack(q[n][h], *(float(*)[E::G])(v + h * E::G));
                if (ragged) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (i + e >= p.d) v[e] = 0.0f;              // padding quantizes to level 0
                }
                uint32_t neg_lo, neg_hi, lo, hi;
                unit_signs<DT>(q[n], neg_lo, neg_hi);
                quantize_unit_bytes<RNG>(v, inv, cap, neg_lo, neg_hi, rw, lo, hi);
                if (m0 + n < p.M) {
                    store_unit_any(p.fmt, lo, hi, (char *)p.lev + (size_t)(m0 + n) * row_bytes, i);
                    const uint32_t bl = lo ^ 0x80808080u, bh = hi ^ 0x80808080u;
                    even[0] += bl & 0x00FF00FFu; odd[0] += (bl >> 8) & 0x00FF00FFu;
                    even[1] += bh & 0x00FF00FFu; odd[1] += (bh >> 8) & 0x00FF00FFu;
                }
            }
        }
        const int bias = 128 * p.M;
        int sum[8];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            sum[4 * k + 0] = (int)(even[k] & 0xFFFFu) - bias;
            sum[4 * k + 1] = (int)(odd[k] & 0xFFFFu) - bias;
            sum[4 * k + 2] = (int)(even[k] >> 16) - bias;
            sum[4 * k + 3] = (int)(odd[k] >> 16) - bias;
        }
        float r[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = __fmul_rn((float)sum[e], c[e]);
        if (!ragged) {
            st_stream256(p.out + i, *(const uint32_t(*)[8])r);
            if (p.S != nullptr) st_stream256(p.S + i, *(const uint32_t(*)[8])sum);
        } else {
            for (int e = 0; e < 8; ++e)
                if (i + e < p.d) {
                    p.out[i + e] = r[e];
                    if (p.S != nullptr) p.S[i + e] = sum[e];
                }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------

int small_max_ctas();

template <int DT, int NORM, int RNG, int IDXB>
static cudaError_t launch_small_multi_one(const SmallParams &p, cudaStream_t st)
{
    static int cache[64] = {};                 // resident CTAs of this instantiation, per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorNotSupported;
    if (cache[dev] == 0) {
        int sms = 0, per_sm = 0, coop = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, small_step_multi_kernel<DT, NORM, RNG, IDXB>, kThreads, 0);
        cache[dev] = coop && sms > 0 && per_sm > 0 ? sms * per_sm : -1;
    }
    if (cache[dev] <= 0) return cudaErrorNotSupported;
    const int64_t want = ((p.d + 7) / 8 + kThreads - 1) / kThreads;
    const int grid = (int)min((int64_t)min(cache[dev], small_max_ctas()), max(want, (int64_t)1));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, small_step_multi_kernel<DT, NORM, RNG, IDXB>, p);
}

template <int DT, int NORM>
static cudaError_t launch_small_multi_idx(const SmallParams &p, int rng_bits, int idx_bits, cudaStream_t st)
{
    if (rng_bits == 32) {
        switch (idx_bits) {
        case 1: return launch_small_multi_one<DT, NORM, 32, 1>(p, st);
        case 2: return launch_small_multi_one<DT, NORM, 32, 2>(p, st);
        case 4: return launch_small_multi_one<DT, NORM, 32, 4>(p, st);
        default: return launch_small_multi_one<DT, NORM, 32, 8>(p, st);
        }
    }
    switch (idx_bits) {
    case 1: return launch_small_multi_one<DT, NORM, 16, 1>(p, st);
    case 2: return launch_small_multi_one<DT, NORM, 16, 2>(p, st);
    case 4: return launch_small_multi_one<DT, NORM, 16, 4>(p, st);
    default: return launch_small_multi_one<DT, NORM, 16, 8>(p, st);
    }
}

cudaError_t launch_small_step_multi(const uq_layout &L, const void *g, int norm, const ScaleSet &scales, int idx_bits,
                                    uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev, float *out,
                                    int32_t *S, uint32_t *status, void *workspace, cudaStream_t st)
{
    SmallParams p;
    p.g = g; p.lev = lev; p.idx = idx; p.W = W; p.out = out; p.S = S; p.status = status;
    p.counter = (uint32_t *)workspace;
    p.part = (double *)((char *)workspace + kSmallHeader);
    p.d = L.d; p.stride = L.worker_stride; p.coord0 = L.coord0; p.M = L.M; p.worker0 = L.worker0;
    p.s = scales.s[0]; p.fmt = fmt; p.scales = scales;
    p.key = philox_key(seed);
    if (L.dtype == UQ_F32)
        return norm == UQ_NORM_L2 ? launch_small_multi_idx<UQ_F32, UQ_NORM_L2>(p, rng_bits, idx_bits, st)
                                  : launch_small_multi_idx<UQ_F32, UQ_NORM_LINF>(p, rng_bits, idx_bits, st);
    return norm == UQ_NORM_L2 ? launch_small_multi_idx<UQ_BF16, UQ_NORM_L2>(p, rng_bits, idx_bits, st)
                              : launch_small_multi_idx<UQ_BF16, UQ_NORM_LINF>(p, rng_bits, idx_bits, st);
}

}  // namespace uq
