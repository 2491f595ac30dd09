// Stochastic quantization of every worker's gradient to small signed integers:
// Q_s (Section "QSGDMaxNorm Quantization", Algorithm 1 line "Quantize gradient") and
// Q_{s_} with the shared per-coordinate scale (Section "QSGDMaxNormMultiScale Quantization",
// Algorithm 2 line "Quantize with s*").
//
// One streaming pass: a thread owns units of 8 consecutive coordinates (32 B of fp32 or 16 B of
// bf16 in; 8 B of int8, 6 B of two-plane 6-bit, 4 B of packed 4-bit or 2 B of packed 2-bit levels
// out); a CTA owns one tile of coordinates and takes the M workers' rows of it one after the other.
// What does not depend on the worker is then done once per tile instead of once per worker: the
// segment lookup, the division s / W, the per-coordinate factors s_k / W of the shared scale
// indices (one index load and eight shuffles per unit), and the first two rounds of the Philox
// block, whose counter differs between workers only in one word.  The work done for worker m
// reads only g^m plus the agreed values W and idx.
#pragma once
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
    uint32_t groups;          // CTAs per tile: ceil(M / kWorkerGroup)
    float cap;                // (float) of the smallest scale: the largest level
    ScaleSet scales;          // single-scale: every entry is s
    PhiloxKey key;            // the ten round keys of the seed
    uint32_t blk_hi;          // high word of the Philox block numbers the table below was made for
    PhiloxWorkerPart wpart[UQ_MAX_WORKERS];   // per-worker words of the first two Philox rounds (row m)
};

constexpr int kWorkerGroup = 8;   // workers that one CTA takes through a tile

// Launch shape per variant, from sweeps on B200: a thread owns UNITS units of 8 coordinates of the
// tile, and at least MIN_CTAS CTAs share an SM (which caps the registers per thread).
template <int DT, int RNG> struct EncodeShape {
    static constexpr int UNITS = DT == UQ_BF16 ? 2 : 1;                       // 32 B per thread and worker in flight
    static constexpr int MIN_CTAS = (DT == UQ_BF16 && RNG == 32) ? 3 : 4;
    static constexpr int TILE = kThreads * UNITS * 8;
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
    using S = EncodeShape<DT, RNG>;
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

// The slow forms of a whole tile, workers m0 .. m1 - 1: the ragged last tile, a tile whose Philox block
// numbers leave the launch's high word, or 16-bit draws with a factor too small for the saturating
// form (j < 0: per-coordinate lookup), and a full tile crossed by segment boundaries (j = its first
// segment).  One out-of-line call keeps their registers out of the straight-line path.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_tile_slow(const EncodeParams &p, int64_t t0, int64_t t1, int j, int m0, int m1)
{
    for (int m = m0; m < m1; ++m) {
        if (j < 0) encode_span_general<DT, FMT, RNG, IDXB>(p, m, t0, t1, threadIdx.x, kThreads);
        else encode_tile_mixed<DT, FMT, RNG, IDXB>(p, m, t0, j);
    }
}

// State of a tile that does not depend on the worker.
template <int DT, int FMT, int RNG, int IDXB> struct TileState {
    using E = Elem<DT>;
    using S = EncodeShape<DT, RNG>;
    static constexpr int U = S::UNITS;
    static constexpr int H = 8 / E::G;                           // 16-byte loads per unit
    static constexpr int BPU = RNG == 32 ? 2 : 1;                // Philox blocks per unit
    float inv[U][8];                  // factor of every coordinate (divided by 256 for 16-bit draws)
    PhiloxBlockPart blk[U * BPU];     // worker-independent rounds of the units' Philox blocks
    SatConstants sc;
    const char *gp;                   // my first coordinate in the gradient row that is loaded next
    char *lp, *lp2;                   // and in the level row that is stored next (second plane for 6-bit)
    size_t grow, lrow;                // bytes between rows
};

template <int DT, int FMT, int RNG, int IDXB>
__device__ __forceinline__ void load_units(TileState<DT, FMT, RNG, IDXB> &t,
                                           uint4 (&q)[EncodeShape<DT, RNG>::UNITS][8 / Elem<DT>::G])
{
    using T = TileState<DT, FMT, RNG, IDXB>;
#pragma unroll
    for (int u = 0; u < T::U; ++u)
#pragma unroll
        for (int h = 0; h < T::H; ++h)
            q[u][h] = ld_stream(t.gp + (u * kThreads * 8 + h * T::E::G) * T::E::BYTES);
    t.gp += t.grow;
}

// Workers m0 .. m0 + G - 1 of the tile, straight-line.  On entry q holds worker m0's units (loaded
// or in flight); while worker m is quantized the units of worker m + 1 are on their way (MORE: also
// those of the worker after the last one of this call).
template <int G, bool MORE, int DT, int FMT, int RNG, int IDXB>
__device__ __forceinline__ void encode_workers(const EncodeParams &p, TileState<DT, FMT, RNG, IDXB> &t, int m0,
                                               uint4 (&q)[EncodeShape<DT, RNG>::UNITS][8 / Elem<DT>::G])
{
    using T = TileState<DT, FMT, RNG, IDXB>;
    using LF = LevelFmt<FMT>;
    constexpr int UB = LF::UB;                                   // bytes of levels per unit: 8, 4 or 2
    constexpr int UB2 = FMT == UQ_FMT_I6P ? 2 : 0;               // and in the second plane of the 6-bit format
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const int m = m0 + k;
        uint4 qn[T::U][T::H];
        if (k + 1 < G || MORE) load_units<DT, FMT, RNG, IDXB>(t, qn);
        uint4 r[T::U * T::BPU];
        philox_join<T::U * T::BPU>(p.key, t.blk, p.wpart[m], r);
#pragma unroll
        for (int u = 0; u < T::U; ++u) {
            float v[8];
#pragma unroll
            for (int h = 0; h < T::H; ++h) T::E::unpack(q[u][h], *(float(*)[T::E::G])(v + h * T::E::G));
            uint32_t neg_lo, neg_hi, lo, hi;
            unit_signs<DT>(q[u], neg_lo, neg_hi);
            if (RNG == 16) {
                quantize_unit_bytes_sat16(v, t.inv[u], t.sc, neg_lo, neg_hi, r[u], lo, hi);
            } else {
                UnitWords<RNG> rw;
                rw.r[0] = r[u * T::BPU]; rw.r[RNG == 32 ? 1 : 0] = r[u * T::BPU + T::BPU - 1];
                quantize_unit_bytes<RNG>(v, t.inv[u], p.cap, neg_lo, neg_hi, rw, lo, hi);
            }
            store_unit<FMT>(lo, hi, t.lp + u * kThreads * UB, t.lp2 + u * kThreads * UB2);
        }
        t.lp += t.lrow;
        if (FMT == UQ_FMT_I6P) t.lp2 += t.lrow;
        if (k + 1 < G || MORE) {
#pragma unroll
            for (int u = 0; u < T::U; ++u)
#pragma unroll
                for (int h = 0; h < T::H; ++h) q[u][h] = qn[u][h];
        }
    }
}

template <int DT, int FMT, int RNG, int IDXB>
__global__ void __launch_bounds__(kThreads, (EncodeShape<DT, RNG>::MIN_CTAS)) encode_kernel(const __grid_constant__ EncodeParams p)
{
    grid_dependency_prologue();
    using T = TileState<DT, FMT, RNG, IDXB>;
    using E = Elem<DT>;
    using S = EncodeShape<DT, RNG>;
    using LF = LevelFmt<FMT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int U = T::U, H = T::H, BPU = T::BPU;
    const int tid = threadIdx.x, lane = tid & 31;
    if (blockIdx.x >= p.main_blocks) {
        // A CTA of the second kind: each warp takes one segment boundary of one worker and, if the
        // boundary lies strictly inside a 256-coordinate row of a full tile, quantizes that row with
        // per-coordinate scales (the tile's own CTA skips it).  Keeping these rows out of the tile
        // CTAs keeps their lifetime short: the slow path no longer holds a whole CTA slot.
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
    // CTAs walk the tiles back to front (see launch_encode); a tile's CTAs take 8 workers each
    const uint32_t rev = p.main_blocks - 1u - blockIdx.x;
    const int64_t tile = (int64_t)(rev / p.groups);
    const int m0 = (int)(rev % p.groups) * kWorkerGroup;
    const int cnt = min(kWorkerGroup, p.M - m0);
    const int64_t t0 = tile * S::TILE;
    const int64_t t1 = min(t0 + (int64_t)S::TILE, p.d);

    // Philox block of the tile's first unit.  The units of a tile add less than 2^12 to it; the
    // straight-line path keeps the high word fixed (the per-worker table of the launch was made for
    // one high word), so a tile in which the low word wraps or whose high word is another one
    // (one launch in 2^35 coordinates) takes the general path like the ragged last tile.
    constexpr int BSH = RNG == 32 ? 2 : 3;                       // coordinates per Philox block, log2
    const uint64_t blk0 = (uint64_t)(p.coord0 >> BSH) + (uint64_t)tile * (uint32_t)(S::TILE >> BSH);
    const bool other_hi = (uint32_t)blk0 > 0xFFFFFFFFu - (uint32_t)(S::TILE >> BSH) || (uint32_t)(blk0 >> 32) != p.blk_hi;
    if (t1 - t0 != S::TILE || other_hi) {
        encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, -1, m0, m0 + cnt);
        return;
    }
    // every warp looks the segment up for itself (no shared memory, no barrier)
    const int j = warp_find_segment(p.seg_off, p.nseg, t0);
    if (segment_end(p.seg_off, p.nseg, j, p.d) < t1) {
        // A segment boundary crosses the tile (at most nseg - 1 tiles): a compact loop over the
        // rows of every worker, kept out of line so that its registers do not weigh on the path below.
        encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, j, m0, m0 + cnt);
        return;
    }
    // the first worker's row and the shared indices
    T t;
    t.grow = (size_t)p.stride * E::BYTES;
    t.lrow = LF::row_bytes(p.stride);
    t.gp = (const char *)p.g + (size_t)m0 * t.grow + ((size_t)t0 + (size_t)tid * 8) * E::BYTES;
    uint4 q[U][H];
    load_units<DT, FMT, RNG, IDXB>(t, q);
    typename IdxBits<IB>::T kbits[U];
    if (MULTI) {
        const uint8_t *ip = p.idx + ((size_t)t0 + (size_t)tid * 8) * IB / 8;
#pragma unroll
        for (int u = 0; u < U; ++u) kbits[u] = IdxBits<IB>::load(ip + u * kThreads * IB);
    }
    // lane k holds s_k / W_j (single-scale: every lane holds s / W_j)
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;    // lane L holds scale L & KMASK
    const float W = __ldg(p.W + j);
    float inv_lane = inv_scale(p.scales.s[lane & KMASK], W);
    if (lane < p.scales.N && not_finite(inv_lane) && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
    if (RNG == 16) {
        if (!sat_form_exact(inv_scale(p.scales.s[0], W))) {        // W beyond 2^100: the plain arithmetic
            encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, -1, m0, m0 + cnt);
            return;
        }
        inv_lane = __fmul_rn(inv_lane, 0.00390625f);
        t.sc = sat_constants(p.cap);
    }
    // the shuffle reads its source lane modulo 32 and the table repeats every 2^IB lanes (an 8-bit
    // index is below 16), so the index bits need a shift but no mask
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int e = 0; e < 8; ++e)
            t.inv[u][e] = MULTI ? __shfl_sync(0xFFFFFFFFu, inv_lane, (int)(uint32_t)(kbits[u] >> (e * IB))) : inv_lane;
    const uint32_t blk_lo = (uint32_t)blk0 + (uint32_t)tid * BPU;
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int b = 0; b < BPU; ++b) t.blk[u * BPU + b] = philox_block_part(p.key, blk_lo + (uint32_t)(u * kThreads * BPU + b));
    char *lrow0 = (char *)p.lev + (size_t)m0 * t.lrow;
    t.lp = lrow0 + LF::off(t0) + tid * LF::UB;
    t.lp2 = lrow0 + LF::off2(t0, p.stride) + tid * (FMT == UQ_FMT_I6P ? 2 : 0);

    // The workers of the group straight-line, with no loop around them: all 8, or (the last group
    // of a job whose M is not a multiple of 8) 4, 2 and 1 of them as the count's bits say.
    if (cnt == kWorkerGroup) {
        encode_workers<kWorkerGroup, false, DT, FMT, RNG, IDXB>(p, t, m0, q);
        return;
    }
    int m = m0;
    if (cnt & 4) {
        if (cnt & 3) encode_workers<4, true, DT, FMT, RNG, IDXB>(p, t, m, q);
        else encode_workers<4, false, DT, FMT, RNG, IDXB>(p, t, m, q);
        m += 4;
    }
    if (cnt & 2) {
        if (cnt & 1) encode_workers<2, true, DT, FMT, RNG, IDXB>(p, t, m, q);
        else encode_workers<2, false, DT, FMT, RNG, IDXB>(p, t, m, q);
        m += 2;
    }
    if (cnt & 1) encode_workers<1, false, DT, FMT, RNG, IDXB>(p, t, m, q);
}

template <int DT, int FMT, int RNG, int IDXB>
static cudaError_t launch(EncodeParams p, cudaStream_t st)
{
    using S = EncodeShape<DT, RNG>;
    p.ntiles = (p.d + S::TILE - 1) / S::TILE;
    p.groups = (uint32_t)((p.M + kWorkerGroup - 1) / kWorkerGroup);
    int64_t blocks = p.ntiles * p.groups;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    p.main_blocks = (uint32_t)blocks;
    if (p.seg_off != nullptr && p.nseg > 1) blocks += (int64_t)((p.nseg - 1 + kWarps - 1) / kWarps) * p.M;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    constexpr int BSH = RNG == 32 ? 2 : 3;
    p.blk_hi = (uint32_t)((uint64_t)(p.coord0 >> BSH) >> 32);
    for (int m = 0; m < UQ_MAX_WORKERS; ++m)
        p.wpart[m] = philox_worker_part(p.key, p.blk_hi, (uint32_t)(p.worker0 + (m < p.M ? m : 0)));
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

// All wire formats and index widths of one element type and draw width (one translation unit
// each, so that the variants build in parallel).
template <int DT, int RNG>
static cudaError_t dispatch_fmt(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st)
{
    if (fmt == UQ_FMT_I8) return dispatch_idx<DT, UQ_FMT_I8, RNG>(p, idx_bits, st);
    if (fmt == UQ_FMT_I4X2) return dispatch_idx<DT, UQ_FMT_I4X2, RNG>(p, idx_bits, st);
    if (fmt == UQ_FMT_I2X4) return dispatch_idx<DT, UQ_FMT_I2X4, RNG>(p, idx_bits, st);
    return dispatch_idx<DT, UQ_FMT_I6P, RNG>(p, idx_bits, st);
}

cudaError_t launch_encode_f32_r16(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st);
cudaError_t launch_encode_f32_r32(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st);
cudaError_t launch_encode_bf16_r16(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st);
cudaError_t launch_encode_bf16_r32(const EncodeParams &p, int fmt, int idx_bits, cudaStream_t st);

}  // namespace uq
