// One whole single-scale step in ONE kernel, for gradients so small that the five launches of the
// regular step cost more than the arithmetic (Algorithm 1, lines "MaxAllReduce Norm" to
// "Reconstruct gradient"; one segment, at most 8 workers).
//
// A cooperative grid (every CTA resident at once) walks the coordinates twice with one grid-wide
// barrier in between:
//   phase 1  each thread adds its units (8 coordinates of every worker) into one norm accumulator
//            per worker; a CTA writes its M partials to the scratch
//   barrier  an arrival counter in the scratch (zero when the kernel starts: the caller zeroes the
//            scratch once, the last CTA through the barrier zeroes the counters again); the wait
//            is bounded: a CTA that gives up sets UQ_STATUS_TIMEOUT and returns
//   phase 2  every CTA adds up all partials in the same fixed order (so all of them hold the same
//            bits of W), then each thread takes its units again (they come from L2 now), quantizes
//            the M workers' values, stores the level rows, adds the levels in SIMD lanes and writes
//            the reconstructed average: the levels never come back from memory
// The gradients cross the HBM interface once, the result leaves once.  Levels, sums and the
// reconstruction are bit for bit those of the separate calls given the same W; W itself is summed
// in another fixed order (L2: within one unit in the last place of the regular kernel's).
#include "uq_small.cuh"

namespace uq {

template <int DT, int NORM, int FMT, int RNG>
__global__ void __launch_bounds__(kThreads, 2) small_step_kernel(const __grid_constant__ SmallParams p)
{
    using E = Elem<DT>;
    using LF = LevelFmt<FMT>;
    constexpr int H = 8 / E::G;
    const int tid = threadIdx.x;
    const int64_t nunits = (p.d + 7) >> 3;
    const int64_t u0 = (int64_t)blockIdx.x * kThreads + tid, ustep = (int64_t)gridDim.x * kThreads;
    float W;
    if (!small_agree<DT, NORM>(p, W)) return;

    // ---- phase 2b: quantize every worker's unit, add the levels, reconstruct
    float inv[8];
    {
        const float f = inv_scale(p.s, W);
#pragma unroll
        for (int e = 0; e < 8; ++e) inv[e] = f;
    }
    const float cap = (float)p.s;
    const float c = __fdiv_rn(W, __fmul_rn((float)p.s, (float)p.M));      // W / ((float)s * (float)M)
    const size_t row_bytes = LF::row_bytes(p.stride);
    constexpr int G = 2;                                                   // workers whose loads are in flight together
    for (int64_t u = u0; u < nunits; u += ustep) {
        const int64_t i = u << 3;
        const char *col = (const char *)p.g + (size_t)i * E::BYTES;
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        const uint32_t blk_lo = (uint32_t)blk, blk_hi = (uint32_t)(blk >> 32);
        const bool ragged = i + 8 > p.d;
        uint32_t even[2] = {0u, 0u}, odd[2] = {0u, 0u};                    // level sums, biased by 128, in 16-bit lanes
        for (int m0 = 0; m0 < p.M; m0 += G) {
            uint4 q[G][H];
#pragma unroll
            for (int n = 0; n < G; ++n) {
                const int m = min(m0 + n, p.M - 1);                        // beyond the last worker: a harmless repeat
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
                        if (i + e >= p.d) v[e] = 0.0f;                     // padding quantizes to level 0
                }
                uint32_t neg_lo, neg_hi, lo, hi;
                unit_signs<DT>(q[n], neg_lo, neg_hi);
                quantize_unit_bytes<RNG>(v, inv, cap, neg_lo, neg_hi, rw, lo, hi);
                if (m0 + n < p.M) {
                    char *row = (char *)p.lev + (size_t)(m0 + n) * row_bytes;
                    store_unit<FMT>(lo, hi, row + LF::off(i), row + LF::off2(i, p.stride));
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
        for (int e = 0; e < 8; ++e) r[e] = __fmul_rn((float)sum[e], c);
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

// CTAs of one instantiation that fit the device at once (cooperative launches need the whole
// grid resident); looked up once per device and instantiation.
template <typename K> static int resident_ctas(K kernel, int *cache)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cache[dev] == 0) {
        int sms = 0, per_sm = 0, coop = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0);
        cache[dev] = coop && sms > 0 && per_sm > 0 ? sms * per_sm : -1;
    }
    return cache[dev] > 0 ? cache[dev] : 0;
}

int small_max_ctas() { return 148 * 8 * 2; }          // bound used to size the scratch (twice today's largest part)

size_t small_workspace_bytes() { return kSmallHeader + (size_t)small_max_ctas() * kSmallMaxWorkers * sizeof(double); }

template <int DT, int NORM, int FMT, int RNG>
static cudaError_t launch_small_one(const SmallParams &p0, cudaStream_t st)
{
    static int cache[64] = {};
    SmallParams p = p0;
    const int resident = resident_ctas(small_step_kernel<DT, NORM, FMT, RNG>, cache);
    if (resident <= 0) return cudaErrorNotSupported;
    const int64_t want = ((p.d + 7) / 8 + kThreads - 1) / kThreads;
    const int grid = (int)min((int64_t)min(resident, small_max_ctas()), max(want, (int64_t)1));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, small_step_kernel<DT, NORM, FMT, RNG>, p);
}

template <int DT, int NORM>
static cudaError_t launch_small_fmt(const SmallParams &p, int fmt, int rng_bits, cudaStream_t st)
{
    switch (fmt) {
    case UQ_FMT_I8:
        return rng_bits == 32 ? launch_small_one<DT, NORM, UQ_FMT_I8, 32>(p, st) : launch_small_one<DT, NORM, UQ_FMT_I8, 16>(p, st);
    case UQ_FMT_I4X2:
        return rng_bits == 32 ? launch_small_one<DT, NORM, UQ_FMT_I4X2, 32>(p, st) : launch_small_one<DT, NORM, UQ_FMT_I4X2, 16>(p, st);
    default:
        return rng_bits == 32 ? launch_small_one<DT, NORM, UQ_FMT_I2X4, 32>(p, st) : launch_small_one<DT, NORM, UQ_FMT_I2X4, 16>(p, st);
    }
}

bool small_step_supported(const uq_layout &L, int fmt)
{
    return L.nseg == 1 && L.M <= kSmallMaxWorkers && (fmt == UQ_FMT_I8 || fmt == UQ_FMT_I4X2 || fmt == UQ_FMT_I2X4);
}

cudaError_t launch_small_step(const uq_layout &L, const void *g, int norm, int s, uint64_t seed, int rng_bits, int fmt,
                              float *W, void *lev, float *out, int32_t *S, uint32_t *status, void *workspace,
                              cudaStream_t st)
{
    SmallParams p;
    p.g = g; p.lev = lev; p.idx = nullptr; p.W = W; p.out = out; p.S = S; p.status = status;
    p.fmt = fmt; p.scales = ScaleSet{};
    p.counter = (uint32_t *)workspace;
    p.part = (double *)((char *)workspace + kSmallHeader);
    p.d = L.d; p.stride = L.worker_stride; p.coord0 = L.coord0; p.M = L.M; p.worker0 = L.worker0; p.s = s;
    p.key = philox_key(seed);
    if (L.dtype == UQ_F32)
        return norm == UQ_NORM_L2 ? launch_small_fmt<UQ_F32, UQ_NORM_L2>(p, fmt, rng_bits, st)
                                  : launch_small_fmt<UQ_F32, UQ_NORM_LINF>(p, fmt, rng_bits, st);
    return norm == UQ_NORM_L2 ? launch_small_fmt<UQ_BF16, UQ_NORM_L2>(p, fmt, rng_bits, st)
                              : launch_small_fmt<UQ_BF16, UQ_NORM_LINF>(p, fmt, rng_bits, st);
}

}  // namespace uq
