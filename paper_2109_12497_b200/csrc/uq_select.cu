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
#include "uq_select.cuh"

namespace uq {

struct SelectParams {
    SelectView v;
    uint8_t *idx;
    uint32_t *status;
};

constexpr int kSelectTile = kThreads * 8;

// LEVELS = ceil(log2 N): the per-coordinate search is a bisection over the N thresholds.
template <int DT, int IDXB, int LEVELS>
__global__ void __launch_bounds__(kThreads) select_kernel(const __grid_constant__ SelectParams p)
{
    grid_dependency_prologue();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t i = ((int64_t)blockIdx.x * kThreads + tid) * 8;   // my first coordinate
    const int64_t row0 = i - (int64_t)lane * 8;                     // my warp's first coordinate
    if (row0 >= p.v.d) return;                                      // warp-uniform
    __shared__ int32_t sh_thr[kWarps][2 * UQ_MAX_SCALES];
    const uint64_t packed = select_unit<DT, IDXB, LEVELS>(p.v, i, row0, sh_thr[warp]);
    if (i < p.v.d) store_unit_indices<IDXB>(p.idx, i, packed);
}

// One row only (M = 1: a single worker, or the row of maxima that uq_agree_scale_amax leaves).
// With nothing to combine across workers the general kernel's per-row setup (segment lookup: two
// dependent loads; threshold table: a division and a short search per scale) is all that is left
// per 256 coordinates, and its latency sets the time.  Here a CTA owns kRowUnits * 2048 coordinates;
// it looks the segment up once and, when that segment covers the whole tile (the common case),
// builds the threshold table once per warp for all its rows; a thread's kRowUnits units are all
// in flight together.  A tile that a boundary crosses falls back to the per-row setup.
constexpr int kRowUnits = 8;

template <int DT, int IDXB, int LEVELS>
__global__ void __launch_bounds__(kThreads, 4) select_row_kernel(const __grid_constant__ SelectParams p)
{
    grid_dependency_prologue();
    using E = Elem<DT>;
    constexpr int H = 8 / E::G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t t0 = (int64_t)blockIdx.x * (kSelectTile * kRowUnits);
    const int64_t t1 = min(t0 + (int64_t)kSelectTile * kRowUnits, p.v.d);
    uint4 q[kRowUnits][H];
#pragma unroll
    for (int u = 0; u < kRowUnits; ++u) {
        const int64_t i = t0 + (int64_t)u * kSelectTile + tid * 8;
#pragma unroll
        for (int h = 0; h < H; ++h)
            q[u][h] = i < p.v.d ? ld_stream((const char *)p.v.g + (size_t)(i + h * E::G) * E::BYTES) : make_uint4(0, 0, 0, 0);
    }
    __shared__ int32_t sh_thr[kWarps][2 * UQ_MAX_SCALES];
    const int jt = warp_find_segment(p.v.seg_off, p.v.nseg, t0);
    const bool tile_uniform = segment_end(p.v.seg_off, p.v.nseg, jt, p.v.d) >= t1;
    int j_table = -1;                                               // segment whose thresholds the table holds
    if (tile_uniform) {
        int32_t thr = -1;
        if (lane < p.v.scales.N) thr = pass_threshold(inv_scale_sel(p.v.scales.s[lane], __ldg(p.v.W + jt)), p.v.s_hat);
        sh_thr[warp][lane] = thr;
        __syncwarp();
        j_table = jt;
    }
#pragma unroll
    for (int u = 0; u < kRowUnits; ++u) {
        const int64_t i = t0 + (int64_t)u * kSelectTile + tid * 8;
        const int64_t row0 = i - (int64_t)lane * 8;
        if (row0 >= p.v.d) break;                                     // warp-uniform
        uint32_t amag[8];
        if (DT == UQ_F32) {
            amag[0] = q[u][0].x & 0x7FFFFFFFu; amag[1] = q[u][0].y & 0x7FFFFFFFu;
            amag[2] = q[u][0].z & 0x7FFFFFFFu; amag[3] = q[u][0].w & 0x7FFFFFFFu;
            amag[4] = q[u][H - 1].x & 0x7FFFFFFFu; amag[5] = q[u][H - 1].y & 0x7FFFFFFFu;
            amag[6] = q[u][H - 1].z & 0x7FFFFFFFu; amag[7] = q[u][H - 1].w & 0x7FFFFFFFu;
        } else {
            const uint32_t w[4] = { q[u][0].x & 0x7FFF7FFFu, q[u][0].y & 0x7FFF7FFFu, q[u][0].z & 0x7FFF7FFFu,
                                    q[u][0].w & 0x7FFF7FFFu };
#pragma unroll
            for (int k = 0; k < 4; ++k) { amag[2 * k] = w[k] << 16; amag[2 * k + 1] = w[k] & 0xFFFF0000u; }
        }
        int j0 = jt;
        bool row_uniform = true;
        if (!tile_uniform) {                                        // per-row setup, as in the general kernel
            const int64_t row1 = min(row0 + 256, p.v.d);
            j0 = warp_find_segment(p.v.seg_off, p.v.nseg, row0);
            row_uniform = segment_end(p.v.seg_off, p.v.nseg, j0, p.v.d) >= row1;
            if (row_uniform && j0 != j_table) {
                __syncwarp();
                int32_t thr = -1;
                if (lane < p.v.scales.N) thr = pass_threshold(inv_scale_sel(p.v.scales.s[lane], __ldg(p.v.W + j0)), p.v.s_hat);
                sh_thr[warp][lane] = thr;
                __syncwarp();
                j_table = j0;
            }
        }
        typename std::conditional<IDXB == 8, uint64_t, uint32_t>::type packed = 0;
        if (row_uniform) {
            const int32_t *T = sh_thr[warp];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int32_t a = (int32_t)amag[e];
                int k = 0;
#pragma unroll
                for (int step = 1 << (LEVELS - 1); step >= 1; step >>= 1)
                    if (a <= T[k + step]) k += step;                // k + step < 2^LEVELS <= 16
                if (i + e >= p.v.d) k = 0;                            // padding keeps index 0
                packed |= (decltype(packed))k << (e * IDXB);
            }
        } else if (i < p.v.d) {
            packed = (decltype(packed))select_general(p.v, i, amag, IDXB, j0);
        }
        if (i >= p.v.d) continue;
        if (IDXB == 1) p.idx[i >> 3] = (uint8_t)packed;
        else if (IDXB == 2) *(uint16_t *)(p.idx + (i >> 2)) = (uint16_t)packed;
        else if (IDXB == 4) *(uint32_t *)(p.idx + (i >> 1)) = (uint32_t)packed;
        else *(uint64_t *)(p.idx + i) = packed;
    }
}

template <int DT, int IDXB>
static cudaError_t dispatch_levels(const SelectParams &p, unsigned blocks, cudaStream_t st)
{
    const int N = p.v.scales.N;
    if (N <= 2) launch_k(select_kernel<DT, IDXB, 1>, blocks, kThreads, st, p);
    else if (N <= 4) launch_k(select_kernel<DT, IDXB, 2>, blocks, kThreads, st, p);
    else if (N <= 8) launch_k(select_kernel<DT, IDXB, 3>, blocks, kThreads, st, p);
    else launch_k(select_kernel<DT, IDXB, 4>, blocks, kThreads, st, p);
    return cudaGetLastError();
}

template <int DT>
static cudaError_t dispatch(const SelectParams &p, int idx_bits, cudaStream_t st)
{
    if (p.v.M == 1 && p.v.d > 0) {                                      // one row: the kernel without per-row setup
        const int64_t nb = (p.v.d + kSelectTile * kRowUnits - 1) / (kSelectTile * kRowUnits);
        if (nb > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
        const int N = p.v.scales.N;
        const int lv = N <= 2 ? 1 : N <= 4 ? 2 : N <= 8 ? 3 : 4;
#define UQ_ROW(IB, LV) launch_k(select_row_kernel<DT, IB, LV>, (unsigned)nb, kThreads, st, p)
        switch (idx_bits * 8 + lv) {
        case 1 * 8 + 1: UQ_ROW(1, 1); break;
        case 2 * 8 + 1: UQ_ROW(2, 1); break;
        case 2 * 8 + 2: UQ_ROW(2, 2); break;
        case 4 * 8 + 1: UQ_ROW(4, 1); break;
        case 4 * 8 + 2: UQ_ROW(4, 2); break;
        case 4 * 8 + 3: UQ_ROW(4, 3); break;
        case 4 * 8 + 4: UQ_ROW(4, 4); break;
        case 8 * 8 + 1: UQ_ROW(8, 1); break;
        case 8 * 8 + 2: UQ_ROW(8, 2); break;
        case 8 * 8 + 3: UQ_ROW(8, 3); break;
        default: UQ_ROW(8, 4); break;
        }
#undef UQ_ROW
        return cudaGetLastError();
    }
    const int64_t blocks = (p.v.d + kSelectTile - 1) / kSelectTile;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (idx_bits == 1) { launch_k(select_kernel<DT, 1, 1>, (unsigned)blocks, kThreads, st, p); return cudaGetLastError(); }
    if (idx_bits == 2) return dispatch_levels<DT, 2>(p, (unsigned)blocks, st);
    if (idx_bits == 4) return dispatch_levels<DT, 4>(p, (unsigned)blocks, st);
    return dispatch_levels<DT, 8>(p, (unsigned)blocks, st);
}

cudaError_t launch_select(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          int idx_bits, uint8_t *idx, uint32_t *status, cudaStream_t st)
{
    SelectParams p;
    p.v.g = g; p.idx = idx; p.v.W = W; p.v.seg_off = L.seg_off; p.status = status;
    p.v.d = L.d; p.v.stride = L.worker_stride; p.v.nseg = L.nseg; p.v.M = L.M;
    p.v.s_hat = (float)scales.s[0];
    p.v.scales = scales;
    return L.dtype == UQ_F32 ? dispatch<UQ_F32>(p, idx_bits, st) : dispatch<UQ_BF16>(p, idx_bits, st);
}

// ---------------------------------------------------------------------------------------------
// Scale sharing across processes (Algorithm 2 line "Scale sharing" when the workers are spread
// over several processes): every process has the minimum over its own workers, packed as the
// selector writes it; the shared index is the field-wise minimum over the R packed rows.
// ---------------------------------------------------------------------------------------------

// Field-wise unsigned minimum of two words holding 4, 8, 16 or 32 fields of 8, 4, 2 or 1 bits.
template <int IDXB> __device__ __forceinline__ uint32_t min_fields(uint32_t a, uint32_t b)
{
    if (IDXB == 1) return a & b;
    if (IDXB == 8) return __vminu4(a, b);
    constexpr uint32_t mask = IDXB == 4 ? 0x0F0F0F0Fu : 0x03030303u;
    uint32_t r = 0;
#pragma unroll
    for (int t = 0; t < 8; t += IDXB) r |= __vminu4((a >> t) & mask, (b >> t) & mask) << t;
    return r;
}

template <int IDXB>
__global__ void __launch_bounds__(kThreads) index_min_kernel(const uint8_t *__restrict__ rows, int R, int64_t row_bytes,
                                                             int64_t nwords, uint8_t *__restrict__ idx)
{
    grid_dependency_prologue();
    const int64_t w = (int64_t)blockIdx.x * kThreads + threadIdx.x;      // my 4-byte word
    if (w >= nwords) return;
    uint32_t acc = __ldg((const uint32_t *)rows + w);
    for (int r = 1; r < R; ++r)
        acc = min_fields<IDXB>(acc, __ldg((const uint32_t *)(rows + (size_t)r * (size_t)row_bytes) + w));
    ((uint32_t *)idx)[w] = acc;
}

cudaError_t launch_index_min(const uint8_t *rows, int R, int64_t row_bytes, int64_t nbytes, int idx_bits, uint8_t *idx,
                             cudaStream_t st)
{
    const int64_t nwords = nbytes / 4;
    const int64_t blocks = (nwords + kThreads - 1) / kThreads;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const unsigned nb = (unsigned)blocks;
    if (idx_bits == 1) launch_k(index_min_kernel<1>, nb, kThreads, st, rows, R, row_bytes, nwords, idx);
    else if (idx_bits == 2) launch_k(index_min_kernel<2>, nb, kThreads, st, rows, R, row_bytes, nwords, idx);
    else if (idx_bits == 4) launch_k(index_min_kernel<4>, nb, kThreads, st, rows, R, row_bytes, nwords, idx);
    else launch_k(index_min_kernel<8>, nb, kThreads, st, rows, R, row_bytes, nwords, idx);
    return cudaGetLastError();
}

}  // namespace uq
