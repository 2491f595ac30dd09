// Shared by the one-kernel steps of the two quantizers (uq_small.cu, uq_small_multi.cu): the kernel
// parameters, the bounded grid-wide barrier and the scale agreement in front of it.
#pragma once
#include "uq_device.cuh"
#include "uq_unit.cuh"
#include "uq_norm.cuh"

namespace uq {

constexpr int kSmallMaxWorkers = 8;
constexpr int kSmallHeader = 64;                  // bytes in front of the partials: arrival and departure counters
constexpr uint32_t kSmallSpinLimit = 1u << 20;    // polls of the counter before a CTA gives up (about a second)

struct SmallParams {
    const void *g;
    void *lev;
    uint8_t *idx;             // multi-scale only
    float *W, *out;
    int32_t *S;
    uint32_t *status;
    uint32_t *counter;        // scratch: [0] arrivals, [1] departures
    double *part;             // scratch: [gridDim.x][kSmallMaxWorkers]
    int64_t d, stride, coord0;
    int32_t M, worker0, s, fmt;
    ScaleSet scales;          // multi-scale only; s = scales.s[0] there
    PhiloxKey key;
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Phase 1, the barrier and phase 2a of a one-kernel step: every thread adds its units into one norm
// accumulator per worker, the CTAs exchange their partials through the scratch and every CTA adds
// them up in the same order.  Returns false if the wait at the barrier ran out (the CTA must
// return); otherwise W is the agreed scale, the same bits in every thread of the grid.
// Must be called by all threads of every CTA of a cooperative grid.
template <int DT, int NORM>
__device__ __forceinline__ bool small_agree(const SmallParams &p, float &W_out)
{
    using E = Elem<DT>;
    constexpr int H = 8 / E::G;
    constexpr int MW = kSmallMaxWorkers;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t nunits = (p.d + 7) >> 3;
    const int64_t u0 = (int64_t)blockIdx.x * kThreads + tid, ustep = (int64_t)gridDim.x * kThreads;
    __shared__ double sh[32][MW];
    __shared__ float sh_w;
    __shared__ int sh_fail;

    // ---- phase 1: per-worker norm partials of my units
    Acc<NORM> acc[MW];
    for (int64_t u = u0; u < nunits; u += ustep) {
        const int64_t i = u << 3;
        const char *col = (const char *)p.g + (size_t)i * E::BYTES;
        const int valid = (int)min((int64_t)8, p.d - i);
#pragma unroll
        for (int m = 0; m < MW; ++m) {
            if (m < p.M) {
                float v[8];
#pragma unroll
                for (int h = 0; h < H; ++h)
                    E::unpack(ld_stream(col + ((size_t)m * (size_t)p.stride + h * E::G) * E::BYTES),
                              *(float(*)[E::G])(v + h * E::G));
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < valid) acc[m].add(v[e]);
            }
        }
    }
#pragma unroll
    for (int m = 0; m < MW; ++m) {
        const double w = m < p.M ? warp_reduce<NORM>(acc[m].value()) : 0.0;     // uniform: idle workers cost nothing
        if (lane == 0) sh[warp][m] = w;
    }
    __syncthreads();
    if (tid < MW) {
        double tot = sh[0][tid];
        for (int k = 1; k < kWarps; ++k) tot = combine<NORM>(tot, sh[k][tid]);
        p.part[(size_t)blockIdx.x * MW + tid] = tot;
    }

    // ---- the grid-wide barrier (bounded)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        __threadfence();                  // release: this CTA's partials (ordered before the barrier above) before its arrival
        atomicAdd(p.counter, 1u);
        uint32_t polls = 0;
        int fail = 0;
        while (ld_acquire(p.counter) < gridDim.x) {
            if (++polls > kSmallSpinLimit) { fail = 1; break; }
            __nanosleep(32);
        }
        __threadfence();                  // acquire: the other CTAs' partials after their arrivals
        if (fail) atomicOr(p.status, (uint32_t)UQ_STATUS_TIMEOUT);
        sh_fail = fail;
        // the last CTA to leave the barrier puts both counters back to zero for the next call
        // (every CTA has read its last value of the arrival counter by then)
        if (!fail && atomicAdd(p.counter + 1, 1u) == gridDim.x - 1) {
            p.counter[1] = 0u;
            __threadfence();
            p.counter[0] = 0u;
        }
    }
    __syncthreads();
    if (sh_fail) return false;

    // ---- phase 2a: W from all partials, in an order that depends on the grid size only
    {
        const int m = tid & (MW - 1), part = tid >> 3;             // 32 strided partial sums per worker
        double a = 0.0;
        for (unsigned c0 = part; c0 < gridDim.x; c0 += 32 * 10) {    // ten loads in flight, added in index order
            double v[10];
#pragma unroll
            for (int k = 0; k < 10; ++k) {
                const unsigned c = c0 + 32u * k;
                v[k] = c < gridDim.x ? __ldcg(p.part + (size_t)c * MW + m) : 0.0;     // 0 is neutral for both norms
            }
#pragma unroll
            for (int k = 0; k < 10; ++k) a = combine<NORM>(a, v[k]);
        }
        sh[part][m] = a;
    }
    __syncthreads();
    if (tid < MW) {                                  // thread m: worker m's 32 sums in index order
        double tot = sh[0][tid];
        for (int k = 1; k < 32; ++k) tot = combine<NORM>(tot, sh[k][tid]);
        sh[0][tid] = tot;                            // only thread m touches column m
    }
    __syncthreads();
    if (tid == 0) {
        bool nan = false;
        double top = 0.0;
        for (int m = 0; m < p.M; ++m) {
            const double tot = sh[0][m];
            nan |= tot != tot;
            top = fmax(top, tot);
        }
        float w;
        if (NORM == UQ_NORM_L2) w = nan ? __uint_as_float(0x7FC00000u) : __double2float_rn(sqrt(top));
        else w = __uint_as_float((uint32_t)top);
        sh_w = w;
        if (blockIdx.x == 0) {
            p.W[0] = w;
            uint32_t flags = 0;
            if (not_finite(w)) flags |= UQ_STATUS_NONFINITE;
            if (not_finite(inv_scale(p.s, w))) flags |= UQ_STATUS_SCALE_OVERFLOW;
            if (flags && p.status) atomicOr(p.status, flags);
        }
    }
    __syncthreads();
    W_out = sh_w;
    return true;
}

}  // namespace uq
