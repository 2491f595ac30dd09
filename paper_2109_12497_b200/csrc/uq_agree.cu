// Shared scale W[j] = max_m || g^m on segment j ||   (Algorithm 1, line "MaxAllReduce Norm").
//
// Two launches.  (1) norm_partials: the coordinate axis is cut into fixed tiles of kNormTile
// coordinates; the CTA of (tile t, worker m) reduces every segment that crosses its tile and
// stores one partial per (tile, segment) pair in slot t + j of worker m's scratch row.  Tiles and
// segments are both ordered, so t + j is unique for every pair and the row needs
// ntiles + nseg slots.  (2) norm_finalize: one CTA per segment adds that segment's slots in a
// fixed order, takes the max over workers, and writes W[j].  The summation tree depends only on
// (d, seg_off), never on the grid or on timing, so W is reproducible bit for bit.
#include "uq_device.cuh"
#include "uq_norm.cuh"

namespace uq {

constexpr int kSlab = 32768;       // tiles per grid.y step of the tile-major order (keeps grid.x below 2^31)

template <int DT, int NORM>
__global__ void __launch_bounds__(kThreads, 8)     // 32 registers: eight CTAs per SM keep HBM busy
norm_partials_kernel(const void *__restrict__ g, int64_t d, int64_t stride, int nseg,
                     const int64_t *__restrict__ seg_off, int64_t ntiles, double *__restrict__ part)
{
    grid_dependency_prologue();
    using E = Elem<DT>;
    constexpr int UNITS = kNormTile / (kThreads * E::G);
    constexpr bool TILE_MAJOR = DT == UQ_F32;
    // CTA order, as measured on B200 (see launch): fp32 walks the tiles front to back with the worker
    // varying fastest (grid.x = M * tiles of one slab of kSlab tiles, grid.y = slab); bf16 streams
    // one worker's row front to back before the next worker's (grid.x = tile, grid.y = worker).
    int m;
    int64_t tile;
    if (TILE_MAJOR) {
        const uint32_t M = gridDim.x / (uint32_t)min(ntiles, (int64_t)kSlab);
        m = (int)(blockIdx.x % M);
        tile = (int64_t)blockIdx.y * kSlab + blockIdx.x / M;
        if (tile >= ntiles) return;                              // the last slab may be ragged
    } else {
        tile = blockIdx.x;
        m = blockIdx.y;
    }
    const int64_t t0 = tile * kNormTile;
    const int64_t t1 = min(t0 + (int64_t)kNormTile, d);
    const char *row = (const char *)g + (size_t)m * (size_t)stride * E::BYTES;
    double *prow = part + (size_t)m * (size_t)(ntiles + nseg);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // The tile's vector loads (the row is padded, so a 16-byte load that starts before d is
    // legal) are issued before the segment lookup when they fit few registers (bf16: 4 loads),
    // after it otherwise (fp32: 8 loads; the lookup is two dependent loads for up to 1024
    // segments, hidden by the other resident CTAs).
    constexpr bool LOADS_FIRST = UNITS <= 4;
    uint4 q[UNITS];
    if (LOADS_FIRST) {
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            const int64_t i = t0 + (int64_t)(u * kThreads + tid) * E::G;
            q[u] = i < t1 ? ld_stream(row + i * E::BYTES) : make_uint4(0, 0, 0, 0);
        }
    }
    const int j0 = warp_find_segment(seg_off, nseg, t0);
    if (segment_end(seg_off, nseg, j0, d) >= t1) {
        // the whole tile lies in segment j0: one block reduction in a fixed order
        if (!LOADS_FIRST) {
#pragma unroll
            for (int u = 0; u < UNITS; ++u) {
                const int64_t i = t0 + (int64_t)(u * kThreads + tid) * E::G;
                q[u] = i < t1 ? ld_stream(row + i * E::BYTES) : make_uint4(0, 0, 0, 0);
            }
        }
        Acc<NORM> acc;
        if (LOADS_FIRST && t1 - t0 == kNormTile) {    // full bf16 tile: no per-element bounds (for
                                                      // fp32 the unguarded form costs 2.5x the registers)
#pragma unroll
            for (int u = 0; u < UNITS; ++u) {
                float v[E::G];
                E::unpack(q[u], v);
#pragma unroll
                for (int e = 0; e < E::G; ++e) acc.add(v[e]);
            }
        } else {
#pragma unroll
            for (int u = 0; u < UNITS; ++u) {
                // elements of this unit that are data (the row's padding beyond d is not)
                const int valid = (int)min((int64_t)E::G, t1 - (t0 + (int64_t)(u * kThreads + tid) * E::G));
                float v[E::G];
                E::unpack(q[u], v);
#pragma unroll
                for (int e = 0; e < E::G; ++e)
                    if (e < valid) acc.add(v[e]);
            }
        }
        __shared__ double sh[kWarps];
        double w = warp_reduce<NORM>(acc.value());
        if (lane == 0) sh[warp] = w;
        __syncthreads();
        if (tid == 0) {
            double tot = sh[0];
#pragma unroll
            for (int k = 1; k < kWarps; ++k) tot = combine<NORM>(tot, sh[k]);
            prow[tile + j0] = tot;
        }
    } else {
        norm_mixed_tile<DT, NORM>(row, prow, tile, t0, t1, d, nseg, seg_off);
    }
}

template <int NORM>
__global__ void __launch_bounds__(kThreads)
norm_finalize_kernel(const double *__restrict__ part, int M, int64_t d, int nseg,
                     const int64_t *__restrict__ seg_off, int64_t ntiles, float *__restrict__ W,
                     uint32_t *__restrict__ status, int tile_coords)       // tile_coords: coordinates per partial
{
    grid_dependency_prologue();
    const int j = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int64_t a = seg_off ? __ldg(seg_off + j) : 0;
    int64_t b = seg_off ? __ldg(seg_off + j + 1) : d;
    const bool bad = a < 0 || b > d || a > b || (j == 0 && a != 0) || (j == nseg - 1 && b != d);
    a = min(max(a, (int64_t)0), d);
    b = min(max(b, a), d);

    double best = 0.0;
    if (a < b) {
        const int64_t first = a / tile_coords, last = (b - 1) / tile_coords;
        for (int m = warp; m < M; m += kWarps) {
            const double *prow = part + (size_t)m * (size_t)(ntiles + nseg) + j;
            double acc = 0.0;
            for (int64_t t = first + lane; t <= last; t += 32) acc = combine<NORM>(acc, prow[t]);
            const double r = warp_reduce<NORM>(acc);
            best = (r != r || best != best) ? r + best : fmax(best, r);   // keep a NaN alive
        }
    }
    __shared__ double sh[kWarps];
    if (lane == 0) sh[warp] = best;
    __syncthreads();
    if (tid == 0) {
        // fmax drops NaN, so look for it explicitly
        bool nan = false;
        double top = 0.0;
        for (int k = 0; k < kWarps; ++k) { nan |= sh[k] != sh[k]; top = fmax(top, sh[k]); }
        float w;
        if (NORM == UQ_NORM_L2) w = nan ? __uint_as_float(0x7FC00000u) : __double2float_rn(sqrt(top));
        else w = __uint_as_float((uint32_t)top);
        W[j] = w;
        uint32_t flags = 0;
        if ((__float_as_uint(w) & 0x7F800000u) == 0x7F800000u) flags |= UQ_STATUS_NONFINITE;
        if (bad) flags |= UQ_STATUS_BAD_SEGMENTS;
        if (flags && status) atomicOr(status, flags);
    }
}

template <int DT, int NORM>
static cudaError_t launch(const uq_layout &L, const void *g, float *W, uint32_t *status, double *part,
                          int64_t ntiles, cudaStream_t st)
{
    if (L.d > 0) {
        if (ntiles > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
        // fp32: tile-major order is 5 % faster on the layer-segmented workloads and neutral on the
        // one-segment ones; bf16: it is 20 % slower than worker-major order
        dim3 grid((unsigned)ntiles, (unsigned)L.M);
        if (DT == UQ_F32)
            grid = dim3((unsigned)L.M * (unsigned)min(ntiles, (int64_t)kSlab), (unsigned)((ntiles + kSlab - 1) / kSlab));
        launch_k(norm_partials_kernel<DT, NORM>, grid, kThreads, st, g, L.d, L.worker_stride, L.nseg,
                                                                 L.seg_off, ntiles, part);
    }
    launch_k(norm_finalize_kernel<NORM>, L.nseg, kThreads, st, part, L.M, L.d, L.nseg, L.seg_off, ntiles, W,
                                                          status, kNormTile);
    return cudaGetLastError();
}

int64_t norm_tiles(int64_t d) { return (d + kNormTile - 1) / kNormTile; }

cudaError_t launch_agree_scale(const uq_layout &L, const void *g, int norm, float *W, uint32_t *status,
                               void *workspace, cudaStream_t st)
{
    const int64_t ntiles = norm_tiles(L.d);
    double *part = (double *)workspace;
    if (L.dtype == UQ_F32)
        return norm == UQ_NORM_L2 ? launch<UQ_F32, UQ_NORM_L2>(L, g, W, status, part, ntiles, st)
                                  : launch<UQ_F32, UQ_NORM_LINF>(L, g, W, status, part, ntiles, st);
    return norm == UQ_NORM_L2 ? launch<UQ_BF16, UQ_NORM_L2>(L, g, W, status, part, ntiles, st)
                              : launch<UQ_BF16, UQ_NORM_LINF>(L, g, W, status, part, ntiles, st);
}

}  // namespace uq

// ---------------------------------------------------------------------------------------------
// uq_agree_scale_static: the same computation with the scratch held inside the library
// ---------------------------------------------------------------------------------------------
#include <mutex>

namespace uq { int record_cuda_error(cudaError_t e); }

namespace {

// Scratch for the norm partials, part of the library image: every GPU that loads the library
// holds these bytes until the process exits.  In host code this name is only a handle; the
// device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[UQ_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void *g_scratch_addr[kMaxDevices] = {};      // device address of g_static_scratch, per device ordinal

// Device address of the scratch array on the current device, resolved once per device.
cudaError_t static_scratch(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *addr = nullptr;
        e = cudaGetSymbolAddress(&addr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (addr == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = addr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int uq_agree_scale_static(const uq_layout *layout, const void *g, int norm, float *W,
                                     uint32_t *status, void *stream)
{
    // size first: a layout that cannot fit is refused before CUDA is touched
    const size_t need = uq_workspace_bytes(layout);
    if (need == 0) return UQ_ERR_BAD_ARG;                       // the layout itself is invalid
    if (need > (size_t)UQ_STATIC_SCRATCH_BYTES) return UQ_ERR_WORKSPACE;
    void *scratch = nullptr;
    const cudaError_t e = static_scratch(&scratch);
    if (e != cudaSuccess) return uq::record_cuda_error(e);      // the code is kept for uq_last_cuda_error()
    // the partials are all written before they are read, so nothing in the array needs clearing
    return uq_agree_scale(layout, g, norm, W, status, scratch, (size_t)UQ_STATIC_SCRATCH_BYTES, stream);
}
