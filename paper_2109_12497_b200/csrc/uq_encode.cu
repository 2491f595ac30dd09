// Stochastic quantization of every worker's gradient to small signed integers:
// Q_s (Section "QSGDMaxNorm Quantization", Algorithm 1 line "Quantize gradient") and
// Q_{s_} with the shared per-coordinate scale (Section "QSGDMaxNormMultiScale Quantization",
// Algorithm 2 line "Quantize with s*").
//
// One streaming pass: a thread owns units of 8 consecutive coordinates (32 B of fp32 or 16 B of
// bf16 in; 8 B of int8, 6 B of two-plane 6-bit, 4 B of packed 4-bit or 2 B of packed 2-bit levels
// out); a CTA owns one tile of one worker.
// A worker's CTA reads only that worker's gradient plus the agreed values W and idx.
#include "uq_device.cuh"
#include "uq_unit.cuh"

namespace uq {

struct EncodeParams {
    const void *g;
    void *lev;
    const float *W;
    const int64_t *seg_off;
    const uint8_t *idx;
    uint32_t *status;
    int64_t d, stride;
    int32_t nseg, M;
    int32_t worker0;          // number, in the whole job, of the worker in row 0 (keys the draws)
    int64_t coord0;           // index, in the whole gradient, of coordinate 0 (keys the draws)
    int64_t ntiles;
    uint32_t main_blocks;     // CTAs that own tiles; the CTAs after them own rows crossed by boundaries
    float cap;                // (float) of the smallest scale: the largest level
    ScaleSet scales;          // single-scale: every entry is s
    PhiloxKey key;            // the ten round keys of the seed
};

// Launch shape per variant, from sweeps on B200 over {4, 8} units x {2..5} CTAs per SM: a thread
// owns UNITS units of 8 coordinates and at least MIN_CTAS CTAs share an SM (which caps the
// registers per thread).  -DUQ_ENCODE_UNITS / -DUQ_ENCODE_MIN_CTAS override all variants (sweeps).
template <int DT, bool MULTI> struct EncodeShape {
#if defined(UQ_ENCODE_UNITS) && defined(UQ_ENCODE_MIN_CTAS)
    static constexpr int UNITS = UQ_ENCODE_UNITS, MIN_CTAS = UQ_ENCODE_MIN_CTAS;
#else
    // fp32 multi-scale: the index shuffles want registers and short unit chains -> 4 units, 4 CTAs
    // bf16 multi-scale: 8 units (128 B in flight per thread), 4 CTAs; single-scale: 8 units, 3 CTAs
    static constexpr int UNITS = (DT == UQ_F32 && MULTI) ? 4 : 8;
    static constexpr int MIN_CTAS = MULTI ? 4 : 3;
#endif
    static constexpr int TILE = kThreads * UNITS * 8;
    // 16-bit draws: units whose Philox blocks advance round by round together (one fetch of a round
    // key serves them all).  Measured: helps the bf16 multi-scale variant, costs the others.
#ifdef UQ_PHILOX_GROUP
    static constexpr int PHILOX_GROUP = UQ_PHILOX_GROUP;
#else
    static constexpr int PHILOX_GROUP = (DT == UQ_BF16 && MULTI) ? 2 : 1;
#endif
};

// Coordinates [a, b) of worker m with per-coordinate scale lookup and bounds: the ragged last
// tile and the 256-coordinate rows that a segment boundary crosses.  Thread `who` of `many`
// cooperating threads (whole warps) takes every many-th unit, so a warp owns a row of 256
// consecutive coordinates per round.  The warp looks the row's first segment up together; lane L
// then holds the end and the scale of segment (first + L), and a coordinate's segment is the
// number of ends at or before it, counted with shuffles: no dependent loads per coordinate.
// Rare (a few rows per segment), so kept out of line.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_span_general(const EncodeParams &p, int m, int64_t a, int64_t b, int who, int many)
{
    using E = Elem<DT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    const char *row = (const char *)p.g + (size_t)m * (size_t)p.stride * E::BYTES;
    const int lane = who & 31;
    for (int64_t row0 = a + (int64_t)(who - lane) * 8; row0 < b; row0 += (int64_t)many * 8) {
        const int64_t row1 = min(row0 + 256, b);
        const int j_row = warp_find_segment(p.seg_off, p.nseg, row0);
        const int jl = j_row + lane;
        const int64_t my_end = jl < p.nseg ? segment_end(p.seg_off, p.nseg, jl, p.d) : INT64_MAX;
        const float my_W = __ldg(p.W + min(jl, p.nseg - 1));
        const int64_t i = min(row0 + lane * 8, b - 1);            // lanes beyond b idle but take part in the shuffles
        int seg[8] = {0, 0, 0, 0, 0, 0, 0, 0};                    // segment of each coordinate, relative to j_row
        int nb = 0;
        for (; nb < 32; ++nb) {                                   // warp-uniform loop over the ends inside the row
            const int64_t end = __shfl_sync(0xFFFFFFFFu, my_end, nb);
            if (end >= row1) break;
#pragma unroll
            for (int e = 0; e < 8; ++e) seg[e] += end <= i + e ? 1 : 0;
        }
        float Wc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) Wc[e] = __shfl_sync(0xFFFFFFFFu, my_W, seg[e]);
        if (nb == 32) {                                           // more than 32 segments in one row: walk the table
            int j = j_row;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                j = advance_segment(p.seg_off, p.nseg, j, i + e);
                Wc[e] = __ldg(p.W + j);
            }
        }
        if (row0 + lane * 8 >= b) continue;
        float v[8];
        uint4 q[8 / E::G];
#pragma unroll
        for (int h = 0; h < 8 / E::G; ++h) {
            q[h] = ld_stream(row + (i + h * E::G) * E::BYTES);
            E::unpack(q[h], *(float(*)[E::G])(v + h * E::G));
        }
        uint32_t neg_lo, neg_hi;
        unit_signs<DT>(q, neg_lo, neg_hi);          // the sign of a padding coordinate is harmless: its level is 0
        typename IdxBits<IB>::T kbits = 0;
        if (MULTI) kbits = IdxBits<IB>::load(p.idx + i * IB / 8);
        float inv[8];
        bool overflow = false;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            if (i + e >= p.d) v[e] = 0.0f;                        // padding quantizes to level 0
            const int k = MULTI ? (int)((kbits >> (e * IB)) & ((1u << IB) - 1u)) : 0;
            inv[e] = inv_scale(p.scales.s[k & (UQ_MAX_SCALES - 1)], Wc[e]);
            overflow |= not_finite(inv[e]);
        }
        if (overflow && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        char *lrow = (char *)p.lev + (size_t)m * LevelFmt<FMT>::row_bytes(p.stride);
        quantize_unit<FMT, RNG>(v, inv, p.cap, neg_lo, neg_hi, p.key, (uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)(m + p.worker0),
                                lrow + LevelFmt<FMT>::off(i), lrow + LevelFmt<FMT>::off2(i, p.stride));
    }
}

// A full tile that a segment boundary crosses, all 256 threads: the warps walk their 256-coordinate
// rows one by one.  Lane L takes the end of segment j + L (j = the tile's first segment), so the
// segment of a row is j + (number of ends at or before the row's start): one ballot per row instead
// of a search.  A row that itself contains a boundary is skipped: a CTA of the second kind owns it.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_tile_mixed(const EncodeParams &p, int m, int64_t t0, int j)
{
    using E = Elem<DT>;
    using S = EncodeShape<DT, IDXB != 0>;
    using LF = LevelFmt<FMT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int H = 8 / E::G;
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;
    const int tid = threadIdx.x, lane = tid & 31;
    const int32_t my_scale = p.scales.s[lane & KMASK];
    const int64_t my_end = j + lane < p.nseg ? segment_end(p.seg_off, p.nseg, j + lane, p.d) : INT64_MAX;
    const char *grow = (const char *)p.g + (size_t)m * (size_t)p.stride * E::BYTES;
    char *lrow = (char *)p.lev + (size_t)m * LF::row_bytes(p.stride);
    bool overflow = false;
#pragma unroll 1
    for (int u = 0; u < S::UNITS; ++u) {
        const int64_t r0 = t0 + (int64_t)(u * kThreads + (tid & ~31)) * 8;
        const int cnt = __popc(__ballot_sync(0xFFFFFFFFu, my_end <= r0));
        int jr;
        int64_t end;
        if (cnt < 32) {
            jr = j + cnt;
            end = __shfl_sync(0xFFFFFFFFu, my_end, cnt);
        } else {                                                 // more than 32 segments inside one tile
            jr = warp_find_segment(p.seg_off, p.nseg, r0);
            end = segment_end(p.seg_off, p.nseg, jr, p.d);
        }
        if (end < r0 + 256) continue;                            // warp-uniform
        const float inv_lane = inv_scale(my_scale, __ldg(p.W + jr));
        overflow |= not_finite(inv_lane);
        const int64_t i = r0 + lane * 8;
        uint4 q[H];
        float v[8], inv[8];
#pragma unroll
        for (int h = 0; h < H; ++h) {
            q[h] = ld_stream(grow + (i + h * E::G) * E::BYTES);
            E::unpack(q[h], *(float(*)[E::G])(v + h * E::G));
        }
        typename IdxBits<IB>::T kbits = 0;
        if (MULTI) kbits = IdxBits<IB>::load(p.idx + i * IB / 8);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            inv[e] = MULTI ? __shfl_sync(0xFFFFFFFFu, inv_lane, (int)(uint32_t)(kbits >> (e * IB))) : inv_lane;
        uint32_t neg_lo, neg_hi;
        unit_signs<DT>(q, neg_lo, neg_hi);
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        quantize_unit<FMT, RNG>(v, inv, p.cap, neg_lo, neg_hi, p.key, (uint32_t)blk, (uint32_t)(blk >> 32),
                                (uint32_t)(m + p.worker0), lrow + LF::off(i), lrow + LF::off2(i, p.stride));
    }
    if (overflow && lane < p.scales.N && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
}

template <int DT, int FMT, int RNG, int IDXB>
__global__ void __launch_bounds__(kThreads, (EncodeShape<DT, IDXB != 0>::MIN_CTAS)) encode_kernel(const __grid_constant__ EncodeParams p)
{
    grid_dependency_prologue();
    using E = Elem<DT>;
    using S = EncodeShape<DT, IDXB != 0>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int H = 8 / E::G;                                  // 16-byte loads per unit
    constexpr uint32_t BPU = RNG == 32 ? 2u : 1u;                // Philox blocks per unit
    constexpr int PG = RNG == 16 ? S::PHILOX_GROUP : 1;            // units whose Philox blocks advance together
    const int tid = threadIdx.x, lane = tid & 31;
    if (blockIdx.x >= p.main_blocks) {
        // A CTA of the second kind: each warp takes one segment boundary and, if the boundary lies
        // strictly inside a 256-coordinate row of a full tile, quantizes that row with per-coordinate
        // scales (the tile's own CTA skips it).  Keeping these rows out of the tile CTAs keeps
        // their lifetime short: the slow path no longer holds a whole CTA slot.
        const uint32_t x = blockIdx.x - p.main_blocks;
        const int m = (int)(x % (uint32_t)p.M);
        const int64_t k = 1 + (int64_t)(x / (uint32_t)p.M) * kWarps + (tid >> 5);
        if (k >= p.nseg) return;
        const int64_t b = __ldg(p.seg_off + k), prev = __ldg(p.seg_off + k - 1);
        const int64_t r0 = b & ~(int64_t)255;
        const int64_t full_end = p.d / S::TILE * S::TILE;          // rows beyond belong to the ragged tile's CTA
        if (b <= 0 || b == r0 || r0 >= full_end) return;           // not strictly inside a row of a full tile
        if (prev > r0 && prev <= b) return;                        // an earlier boundary in the same row takes it
        encode_span_general<DT, FMT, RNG, IDXB>(p, m, r0, r0 + 256, lane, 32);
        return;
    }
    // CTAs walk the tiles back to front with the worker varying fastest (see launch_encode)
    const uint32_t rev = p.main_blocks - 1u - blockIdx.x;
    const int m = (int)(rev % (uint32_t)p.M);
    const int64_t tile = rev / (uint32_t)p.M;
    const int64_t t0 = tile * S::TILE;
    const int64_t t1 = min(t0 + (int64_t)S::TILE, p.d);

    // Philox block of the tile's first unit.  The units of a tile add less than 2^13 to it; the
    // straight-line path keeps the high word fixed, so the one tile in 2^35 coordinates in which
    // the low word wraps takes the general path (64-bit block numbers) like the ragged last tile.
    constexpr int BSH = RNG == 32 ? 2 : 3;                       // coordinates per Philox block, log2
    const uint64_t blk0 = (uint64_t)(p.coord0 >> BSH) + (uint64_t)tile * (uint32_t)(S::TILE >> BSH);
    const bool wraps = (uint32_t)blk0 > 0xFFFFFFFFu - (uint32_t)(S::TILE >> BSH);
    if (t1 - t0 != S::TILE || wraps) {
        encode_span_general<DT, FMT, RNG, IDXB>(p, m, t0, t1, tid, kThreads);
        return;
    }
    // issue the loads of the full tile first; the segment lookup overlaps with them
    const char *gp = (const char *)p.g + ((size_t)m * (size_t)p.stride + (size_t)t0 + (size_t)tid * 8) * E::BYTES;
    const uint8_t *ip = MULTI ? p.idx + ((size_t)t0 + (size_t)tid * 8) * IB / 8 : nullptr;
    uint4 q[S::UNITS][H];
    typename IdxBits<IB>::T kbits[S::UNITS];
#pragma unroll
    for (int u = 0; u < S::UNITS; ++u) {
#pragma unroll
        for (int h = 0; h < H; ++h) q[u][h] = ld_stream(gp + (u * kThreads * 8 + h * E::G) * E::BYTES);
        if (MULTI) kbits[u] = IdxBits<IB>::load(ip + u * kThreads * IB);
    }
    // every warp looks the segment up for itself (no shared memory, no barrier): once for the
    // tile if one segment covers it, else once per 256-coordinate row of the warp.
    // lane k holds s_k / W_j (single-scale: every lane holds s / W_j)
    const int j = warp_find_segment(p.seg_off, p.nseg, t0);
    const bool tile_uniform = segment_end(p.seg_off, p.nseg, j, p.d) >= t1;
    if (!tile_uniform) {
        // A segment boundary crosses the tile (at most nseg - 1 tiles per worker): a compact loop
        // over the rows, kept out of line so that its registers do not weigh on the path below.
        // (The loads issued above are dropped; that loop fetches its rows again, from L2.)
        encode_tile_mixed<DT, FMT, RNG, IDXB>(p, m, t0, j);
        return;
    }
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;    // lane L holds scale L & KMASK
    const float inv_lane = inv_scale(p.scales.s[lane & KMASK], __ldg(p.W + j));
    bool overflow = false;                                       // some s_k / W is not finite
    if (MULTI) overflow = not_finite(inv_lane);

    const uint32_t blk_hi = (uint32_t)(blk0 >> 32);
    const uint32_t blk_lo = (uint32_t)blk0 + (uint32_t)tid * BPU;
    using LF = LevelFmt<FMT>;
    constexpr int UB = LF::UB;                                   // bytes of levels per unit: 8, 4 or 2
    constexpr int UB2 = FMT == UQ_FMT_I6P ? 2 : 0;               // and in the second plane of the 6-bit format
    char *lrow = (char *)p.lev + (size_t)m * LF::row_bytes(p.stride);
    char *lp = lrow + LF::off(t0) + tid * UB;
    char *lp2 = lrow + LF::off2(t0, p.stride) + tid * UB2;
    // One straight-line pass over all units, so the compiler can interleave them.
#pragma unroll
    for (int u0 = 0; u0 < S::UNITS; u0 += PG) {
        // the random words of PG units together (16-bit draws: one Philox block per unit)
        UnitWords<RNG> rw[PG];
        if (RNG == 16) {
            uint32_t b[PG];
            uint4 r[PG];
#pragma unroll
            for (int n = 0; n < PG; ++n) b[n] = blk_lo + (u0 + n) * kThreads * BPU;
            philox4x32_10_xN<PG>(p.key, b, blk_hi, (uint32_t)(m + p.worker0), r);
#pragma unroll
            for (int n = 0; n < PG; ++n) rw[n].r[0] = r[n];
        } else {
            rw[0] = unit_words<RNG>(p.key, blk_lo + u0 * kThreads * BPU, blk_hi, (uint32_t)(m + p.worker0));
        }
#pragma unroll
        for (int n = 0; n < PG; ++n) {
            const int u = u0 + n;
            // where the finiteness check sits is a measured choice: ahead of the loop for the
            // multi-scale variants (1.5 % faster on bf16), inside it for the single-scale ones (the
            // hoisted form compiles to a 3-7 % slower kernel there)
            if (!MULTI) overflow |= not_finite(inv_lane);
            float v[8], inv[8];
#pragma unroll
            for (int h = 0; h < H; ++h) E::unpack(q[u][h], *(float(*)[E::G])(v + h * E::G));
            // the shuffle reads its source lane modulo 32 and the table repeats every 2^IB lanes (an
            // 8-bit index is below 16), so the index bits need a shift but no mask
#pragma unroll
            for (int e = 0; e < 8; ++e)
                inv[e] = MULTI ? __shfl_sync(0xFFFFFFFFu, inv_lane, (int)(uint32_t)(kbits[u] >> (e * IB))) : inv_lane;
            uint32_t neg_lo, neg_hi;
            unit_signs<DT>(q[u], neg_lo, neg_hi);
            quantize_unit_words<FMT, RNG>(v, inv, p.cap, neg_lo, neg_hi, rw[n], lp + u * kThreads * UB,
                                          lp2 + u * kThreads * UB2);
        }
    }
    if (overflow && lane < p.scales.N && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
}

template <int DT, int FMT, int RNG, int IDXB>
static cudaError_t launch(EncodeParams p, cudaStream_t st)
{
    using S = EncodeShape<DT, IDXB != 0>;
    p.ntiles = (p.d + S::TILE - 1) / S::TILE;
    int64_t blocks = p.ntiles * p.M;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    p.main_blocks = (uint32_t)blocks;
    if (p.seg_off != nullptr && p.nseg > 1) blocks += (int64_t)((p.nseg - 1 + kWarps - 1) / kWarps) * p.M;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    launch_k(encode_kernel<DT, FMT, RNG, IDXB>, (unsigned)blocks, kThreads, st, p);
    return cudaGetLastError();
}

template <int DT, int FMT, int RNG>
static cudaError_t dispatch_idx(const EncodeParams &p, int idx_bits, cudaStream_t st)
{
    switch (idx_bits) {
    case 0: return launch<DT, FMT, RNG, 0>(p, st);
    case 1: return launch<DT, FMT, RNG, 1>(p, st);
    case 2: return launch<DT, FMT, RNG, 2>(p, st);
    case 4: return launch<DT, FMT, RNG, 4>(p, st);
    default: return launch<DT, FMT, RNG, 8>(p, st);
    }
}

template <int DT>
static cudaError_t dispatch_fmt(const EncodeParams &p, int fmt, int rng_bits, int idx_bits, cudaStream_t st)
{
    if (fmt == UQ_FMT_I8)
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I8, 32>(p, idx_bits, st)
                              : dispatch_idx<DT, UQ_FMT_I8, 16>(p, idx_bits, st);
    if (fmt == UQ_FMT_I4X2)
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I4X2, 32>(p, idx_bits, st)
                              : dispatch_idx<DT, UQ_FMT_I4X2, 16>(p, idx_bits, st);
    if (fmt == UQ_FMT_I2X4)
        return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I2X4, 32>(p, idx_bits, st)
                              : dispatch_idx<DT, UQ_FMT_I2X4, 16>(p, idx_bits, st);
    return rng_bits == 32 ? dispatch_idx<DT, UQ_FMT_I6P, 32>(p, idx_bits, st)
                          : dispatch_idx<DT, UQ_FMT_I6P, 16>(p, idx_bits, st);
}

// idx_bits == 0 selects the single-scale quantizer (scales = {s}).
cudaError_t launch_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                          uint32_t *status, cudaStream_t st)
{
    EncodeParams p;
    p.g = g; p.lev = lev; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.status = status;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M; p.worker0 = L.worker0; p.coord0 = L.coord0;
    p.key = philox_key(seed);
    // CTA order (set in the kernel): the tiles are walked back to front with the worker varying fastest.  The
    // kernel before this one in a step (agree-scale or the selector) ends on the high tiles, so
    // part of what is read first is still in L2; all M workers of a tile run together, which
    // keeps one copy of the shared index tile in L2 and spreads the streams over the memory
    // channels (measured faster than walking worker by worker); and the kernel ends on the lowest
    // tiles, where the aggregation starts.
    p.cap = (float)scales.s[0];
    p.scales = scales;
    return L.dtype == UQ_F32 ? dispatch_fmt<UQ_F32>(p, fmt, rng_bits, idx_bits, st)
                             : dispatch_fmt<UQ_BF16>(p, fmt, rng_bits, idx_bits, st);
}

}  // namespace uq
