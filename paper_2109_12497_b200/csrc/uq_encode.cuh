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
//
// Decode mode (int8 levels, 16-bit draws, M <= 8, so that one CTA sees every worker of its tile; with
// 32-bit draws the encoder is bound by its arithmetic and the sums cost what the saved read gains,
// measured, so there the two kernels stay): the CTA also adds
// the workers' levels up as it goes and writes the reconstructed average (Algorithm 1 / 2, lines
// "AllReduce gradients" and "Reconstruct gradient") beside the level rows, which then need not be
// read back by the aggregation kernel.  Bit for bit what uq_decode makes of the same levels.
#pragma once
#include "uq_device.cuh"
#include "uq_select.cuh"
#include "uq_unit.cuh"

namespace uq {

struct EncodeParams {
    SelectView v;             // g, W, seg_off, d, stride, nseg, M, scales (single-scale: every entry is s) and
                              // s_hat = (float) of the smallest scale: the largest level
    void *lev;
    float *out;               // decode mode: the reconstructed average [d]; else unused
    uint8_t *idx;             // shared scale indices: read, or (select) written by this launch
    uint32_t *status;
    int32_t select;           // multi-scale: 1 = find the shared indices here instead of reading them
    int32_t worker0;          // number, in the whole job, of the worker in row 0 (keys the draws)
    int64_t coord0;           // index, in the whole gradient, of coordinate 0 (keys the draws)
    uint32_t row_blocks;      // CTAs that own rows crossed by boundaries: after the tile CTAs, or (decode mode,
                              // where such a CTA takes every worker's row and runs much longer) in front of them
    uint32_t reserved;
    uint32_t main_blocks;     // CTAs that own tiles
    uint32_t groups;          // CTAs per tile: ceil(M / kWorkerGroup)
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
    // decode mode (16-bit draws only) holds the level sums too: at 64 registers the bf16 kernel spills
    static constexpr int MIN_CTAS_DEC = DT == UQ_F32 ? 4 : 3;
    static constexpr int TILE = kThreads * UNITS * 8;
};

// Coordinates [a, b) of worker m with per-coordinate scale lookup and bounds: the ragged last
// tile and the 256-coordinate rows that a segment boundary crosses.  Thread `who` of `many`
// cooperating threads (whole warps) takes every many-th unit, so a warp owns a row of 256
// consecutive coordinates per round.  The warp looks the row's first segment up together; lane L
// then holds the end and the scale of segment (first + L), and a coordinate's segment is the
// number of ends at or before it, counted with shuffles: no dependent loads per coordinate.
// Rare (a few rows per segment), so kept out of line.
// own_idx (select mode, rows owned by a CTA that did not select for them): the warp finds the
// shared indices of its row itself (thr: the warp's 2 * UQ_MAX_SCALES words of shared memory) instead
// of reading them.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_span_general(const EncodeParams &p, int m, int64_t a, int64_t b, int who, int many,
                                                 bool own_idx = false, int32_t *thr = nullptr)
{
    using E = Elem<DT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    const char *row = (const char *)p.v.g + (size_t)m * (size_t)p.v.stride * E::BYTES;
    const int lane = who & 31;
    for (int64_t row0 = a + (int64_t)(who - lane) * 8; row0 < b; row0 += (int64_t)many * 8) {
        const int64_t row1 = min(row0 + 256, b);
        const int j_row = warp_find_segment(p.v.seg_off, p.v.nseg, row0);
        const int jl = j_row + lane;
        const int64_t my_end = jl < p.v.nseg ? segment_end(p.v.seg_off, p.v.nseg, jl, p.v.d) : INT64_MAX;
        const float my_W = __ldg(p.v.W + min(jl, p.v.nseg - 1));
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
                j = advance_segment(p.v.seg_off, p.v.nseg, j, i + e);
                Wc[e] = __ldg(p.v.W + j);
            }
        }
        typename IdxBits<IB>::T kbits = 0;
        if (MULTI && own_idx)                                     // the whole warp takes part
            kbits = (typename IdxBits<IB>::T)select_unit<DT, IB, 4>(p.v, row0 + lane * 8, row0, thr);
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
        if (MULTI && !own_idx)
            kbits = p.select ? IdxBits<IB>::load_written(p.idx + i * IB / 8) : IdxBits<IB>::load(p.idx + i * IB / 8);
        float inv[8];
        bool overflow = false;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            if (i + e >= p.v.d) v[e] = 0.0f;                        // padding quantizes to level 0
            const int k = MULTI ? (int)((kbits >> (e * IB)) & ((1u << IB) - 1u)) : 0;
            inv[e] = inv_scale(p.v.scales.s[k & (UQ_MAX_SCALES - 1)], Wc[e]);
            overflow |= not_finite(inv[e]);
        }
        if (overflow && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        char *lrow = (char *)p.lev + (size_t)m * LevelFmt<FMT>::row_bytes(p.v.stride);
        quantize_unit<FMT, RNG>(v, inv, p.v.s_hat, neg_lo, neg_hi, p.key, (uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)(m + p.worker0),
                                lrow + LevelFmt<FMT>::off(i), lrow + LevelFmt<FMT>::off2(i, p.v.stride));
    }
}

// A full tile that a segment boundary crosses, all 256 threads, workers m0 .. m1 - 1: the warps
// walk their 256-coordinate rows one by one.  Lane L takes the end of segment j + L (j = the
// tile's first segment), so the segment of a row is j + (number of ends at or before the row's
// start): one ballot per row instead of a search.  What a row's workers share (its segment, the
// factors s_k / W, the shared indices) is found once per row; the rows of four workers are in
// flight together.  A row that itself contains a boundary is skipped: a CTA of the second kind
// owns it.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_tile_mixed(const EncodeParams &p, int m0, int m1, int64_t t0, int j)
{
    using E = Elem<DT>;
    using S = EncodeShape<DT, RNG>;
    using LF = LevelFmt<FMT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int H = 8 / E::G;
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;
    constexpr int G = 4;                                         // workers whose rows are loaded together
    const int tid = threadIdx.x, lane = tid & 31;
    const int32_t my_scale = p.v.scales.s[lane & KMASK];
    const int64_t my_end = j + lane < p.v.nseg ? segment_end(p.v.seg_off, p.v.nseg, j + lane, p.v.d) : INT64_MAX;
    const size_t grow = (size_t)p.v.stride * E::BYTES, lrow = LF::row_bytes(p.v.stride);
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
            jr = warp_find_segment(p.v.seg_off, p.v.nseg, r0);
            end = segment_end(p.v.seg_off, p.v.nseg, jr, p.v.d);
        }
        if (end < r0 + 256) continue;                            // warp-uniform
        const float inv_lane = inv_scale(my_scale, __ldg(p.v.W + jr));
        overflow |= not_finite(inv_lane);
        const int64_t i = r0 + lane * 8;
        typename IdxBits<IB>::T kbits = 0;
        if (MULTI) kbits = p.select ? IdxBits<IB>::load_written(p.idx + i * IB / 8) : IdxBits<IB>::load(p.idx + i * IB / 8);
        float inv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e)
            inv[e] = MULTI ? __shfl_sync(0xFFFFFFFFu, inv_lane, (int)(uint32_t)(kbits >> (e * IB))) : inv_lane;
        const uint64_t blk = RNG == 32 ? (uint64_t)((p.coord0 + i) >> 2) : (uint64_t)((p.coord0 + i) >> 3);
        const char *gp = (const char *)p.v.g + (size_t)m0 * grow + (size_t)i * E::BYTES;
        char *lp = (char *)p.lev + (size_t)m0 * lrow;
#pragma unroll 1
        for (int m = m0; m < m1; m += G) {
            uint4 q[G][H];
#pragma unroll
            for (int k = 0; k < G; ++k)
                if (m + k < m1) {
#pragma unroll
                    for (int h = 0; h < H; ++h) q[k][h] = ld_stream(gp + (size_t)k * grow + h * E::G * E::BYTES);
                }
#pragma unroll
            for (int k = 0; k < G; ++k)
                if (m + k < m1) {
                    float v[8];
#pragma unroll
                    for (int h = 0; h < H; ++h) E::unpack(q[k][h], *(float(*)[E::G])(v + h * E::G));
                    uint32_t neg_lo, neg_hi;
                    unit_signs<DT>(q[k], neg_lo, neg_hi);
                    quantize_unit<FMT, RNG>(v, inv, p.v.s_hat, neg_lo, neg_hi, p.key, (uint32_t)blk, (uint32_t)(blk >> 32),
                                            (uint32_t)(m + k + p.worker0), lp + (size_t)k * lrow + LF::off(i),
                                            lp + (size_t)k * lrow + LF::off2(i, p.v.stride));
                }
            gp += G * grow;
            lp += G * lrow;
        }
    }
    if (overflow && lane < p.v.scales.N && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
}

// Decode mode, slow forms: sum and reconstruction of the unit of 8 coordinates at i from the int8
// levels that THIS thread stored for every worker just before (own stores are visible to own loads;
// read around L1), with the segment and the shared index looked up per coordinate.
template <int IDXB>
__device__ __noinline__ void decode_unit_general(const EncodeParams &p, int64_t i, uint64_t kbits_own, bool own_idx)
{
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    if (i >= p.v.d) return;
    int S[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const char *lp = (const char *)p.lev + i;
    for (int m = 0; m < p.v.M; ++m) {
        const uint2 b = __ldcg((const uint2 *)(lp + (size_t)m * (size_t)p.v.stride));
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            S[e] += (int)(int8_t)(b.x >> (8 * e));
            S[4 + e] += (int)(int8_t)(b.y >> (8 * e));
        }
    }
    uint64_t kbits = kbits_own;
    if (MULTI && !own_idx)        // select mode: the CTA stored the tile's indices itself (behind a barrier)
        kbits = (uint64_t)(p.select ? IdxBits<IB>::load_written(p.idx + i * IB / 8) : IdxBits<IB>::load(p.idx + i * IB / 8));
    int j = find_segment(p.v.seg_off, p.v.nseg, i);
    for (int e = 0; e < 8 && i + e < p.v.d; ++e) {
        j = advance_segment(p.v.seg_off, p.v.nseg, j, i + e);
        const int k = MULTI ? (int)((kbits >> (e * IB)) & ((1u << IB) - 1u)) : 0;
        p.out[i + e] = __fmul_rn((float)S[e], decode_factor(__ldg(p.v.W + j), p.v.scales.s[k & (UQ_MAX_SCALES - 1)], p.v.M));
    }
}

// The units of tile [t0, t1) that this thread encoded in a slow form (the same assignment of units to
// threads as encode_span_general and encode_tile_mixed).  mixed: a full tile crossed by boundaries; a
// row that itself contains a boundary was skipped there and is skipped here (a CTA of the second
// kind owns it), every other row lies in one segment, so lane k takes the factor of scale k once
// per row.  Else (ragged tile and the like) everything is looked up per coordinate.
template <int DT, int RNG, int IDXB>
__device__ __noinline__ void decode_tile_slow(const EncodeParams &p, int64_t t0, int64_t t1, bool mixed)
{
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;
    const int lane = threadIdx.x & 31;
    for (int u = 0; u < EncodeShape<DT, RNG>::UNITS; ++u) {
        const int64_t r0 = t0 + (int64_t)(u * kThreads + (threadIdx.x & ~31)) * 8;
        if (r0 >= t1) break;                                         // warp-uniform
        const int64_t i = r0 + lane * 8;
        if (!mixed) {
            if (i < t1) decode_unit_general<IDXB>(p, i, 0, false);
            continue;
        }
        const int jr = warp_find_segment(p.v.seg_off, p.v.nseg, r0);
        if (segment_end(p.v.seg_off, p.v.nseg, jr, p.v.d) < r0 + 256) continue;
        const float c_lane = decode_factor(__ldg(p.v.W + jr), p.v.scales.s[lane & KMASK], p.v.M);
        uint32_t sum[4] = {0u, 0u, 0u, 0u};                          // as in the straight-line path
        const char *lp = (const char *)p.lev + i;
        for (int m = 0; m < p.v.M; ++m) {
            const uint2 b = __ldcg((const uint2 *)(lp + (size_t)m * (size_t)p.v.stride));
            const uint32_t bl = b.x ^ 0x80808080u, bh = b.y ^ 0x80808080u;
            sum[0] += __byte_perm(bl, 0u, 0x4240); sum[1] += __byte_perm(bl, 0u, 0x4341);
            sum[2] += __byte_perm(bh, 0u, 0x4240); sum[3] += __byte_perm(bh, 0u, 0x4341);
        }
        typename IdxBits<IB>::T kbits = 0;
        if (MULTI) kbits = p.select ? IdxBits<IB>::load_written(p.idx + i * IB / 8) : IdxBits<IB>::load(p.idx + i * IB / 8);
        const int bias = 128 * p.v.M;
        uint32_t r[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int S = (int)((sum[(e >> 2) * 2 + (e & 1)] >> (16 * ((e & 3) >> 1))) & 0xFFFFu) - bias;
            const float c = MULTI ? __shfl_sync(0xFFFFFFFFu, c_lane, (int)(uint32_t)(kbits >> (e * IB))) : c_lane;
            r[e] = __float_as_uint(__fmul_rn((float)S, c));
        }
        st_stream256(p.out + i, r);
    }
}

// The slow forms of a whole tile, workers m0 .. m1 - 1: the ragged last tile, a tile whose Philox block
// numbers leave the launch's high word, or 16-bit draws with a factor too small for the saturating
// form (j < 0: per-coordinate lookup), and a full tile crossed by segment boundaries (j = its first
// segment).  One out-of-line call keeps their registers out of the straight-line path.
// In select mode the CTA first finds and stores the shared indices of the whole tile (thr: the
// CTA's kWarps * 2 * UQ_MAX_SCALES words of shared memory); the encoding then reads them back.
template <int DT, int FMT, int RNG, int IDXB>
__device__ __noinline__ void encode_tile_slow(const EncodeParams &p, int64_t t0, int64_t t1, int j, int m0, int m1,
                                              int32_t *thr)
{
    if (IDXB != 0 && p.select) {
        constexpr int IB = IDXB != 0 ? IDXB : 8;
        const int lane = threadIdx.x & 31;
        for (int u = 0; u < EncodeShape<DT, RNG>::UNITS; ++u) {
            const int64_t i = t0 + (int64_t)(u * kThreads + threadIdx.x) * 8;
            const int64_t row0 = i - lane * 8;
            if (row0 >= t1) break;                                   // warp-uniform
            const uint64_t packed = select_unit<DT, IB, 4>(p.v, i, row0, thr + (threadIdx.x >> 5) * 2 * UQ_MAX_SCALES);
            if (i < p.v.d) store_unit_indices<IB>(p.idx, i, packed);
        }
        __syncthreads();                                             // the tile's indices are in memory for all warps
    }
    if (j >= 0) {
        encode_tile_mixed<DT, FMT, RNG, IDXB>(p, m0, m1, t0, j);
        return;
    }
    for (int m = m0; m < m1; ++m) encode_span_general<DT, FMT, RNG, IDXB>(p, m, t0, t1, threadIdx.x, kThreads);
}

// State of a tile that does not depend on the worker.
template <int DT, int FMT, int RNG, int IDXB, bool DEC = false> struct TileState {
    using E = Elem<DT>;
    using S = EncodeShape<DT, RNG>;
    static constexpr int U = S::UNITS;
    static constexpr int H = 8 / E::G;                           // 16-byte loads per unit
    static constexpr int BPU = RNG == 32 ? 2 : 1;                // Philox blocks per unit
    float inv[U][8];                  // factor of every coordinate: / 256 for 16-bit draws, * 2^23 for 32-bit draws
    PhiloxBlockPart blk[U * BPU];     // worker-independent rounds of the units' Philox blocks
    SatConstants sc;                  // 16-bit draws
    float cap23;                      // 32-bit draws: the largest level * 2^23
    uint32_t sum[DEC ? U : 1][4];     // decode mode: the unit's level sums, every level biased by 128, in 16-bit
                                      // lanes: bytes 0, 2 and bytes 1, 3 of the low word, then of the high word
    const char *gp;                   // my first coordinate in the gradient row that is loaded next
    const uint4 *sp;                  // select mode: my slot of that row's copy in shared memory
    char *lp, *lp2;                   // and in the level row that is stored next (second plane for 6-bit)
    size_t grow, lrow;                // bytes between rows
};

template <bool SEL, int DT, int FMT, int RNG, int IDXB, bool DEC>
__device__ __forceinline__ void load_units(TileState<DT, FMT, RNG, IDXB, DEC> &t,
                                           uint4 (&q)[EncodeShape<DT, RNG>::UNITS][8 / Elem<DT>::G])
{
    using T = TileState<DT, FMT, RNG, IDXB, DEC>;
#pragma unroll
    for (int u = 0; u < T::U; ++u)
#pragma unroll
        for (int h = 0; h < T::H; ++h)
            q[u][h] = SEL ? t.sp[(u * T::H + h) * kThreads] : ld_stream(t.gp + (u * kThreads * 8 + h * T::E::G) * T::E::BYTES);
    if (SEL) t.sp += T::U * T::H * kThreads;
    else t.gp += t.grow;
}

// Workers m0 .. m0 + G - 1 of the tile, straight-line.  On entry q holds worker m0's units (loaded
// or in flight); while worker m is quantized the units of worker m + 1 are on their way (MORE: also
// those of the worker after the last one of this call).
template <int G, bool MORE, bool SEL, int DT, int FMT, int RNG, int IDXB, bool DEC>
__device__ __forceinline__ void encode_workers(const EncodeParams &p, TileState<DT, FMT, RNG, IDXB, DEC> &t, int m0,
                                               uint4 (&q)[EncodeShape<DT, RNG>::UNITS][8 / Elem<DT>::G])
{
    using T = TileState<DT, FMT, RNG, IDXB, DEC>;
    using LF = LevelFmt<FMT>;
    constexpr int UB = LF::UB;                                   // bytes of levels per unit: 8, 4 or 2
    constexpr int UB2 = FMT == UQ_FMT_I6P ? 2 : 0;               // and in the second plane of the 6-bit format
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const int m = m0 + k;
        uint4 qn[T::U][T::H];
        if (k + 1 < G || MORE) load_units<SEL>(t, qn);
        uint4 r[T::U * T::BPU];
        philox_join<T::U * T::BPU>(p.key, t.blk, p.wpart[m], r);
#pragma unroll
        for (int u = 0; u < T::U; ++u) {
            float v[8];
#pragma unroll
            for (int h = 0; h < T::H; ++h) T::E::unpack(q[u][h], *(float(*)[T::E::G])(v + h * T::E::G));
            // binary32 to 4 bits: the unit's bytes in even / odd order, which the store merges directly
            constexpr bool EO = FMT == UQ_FMT_I4X2 && DT == UQ_F32;
            uint32_t neg_lo, neg_hi, lo, hi;
            unit_signs<DT, EO>(q[u], neg_lo, neg_hi);
            if (RNG == 16) {
                quantize_unit_bytes_sat16<EO>(v, t.inv[u], t.sc, neg_lo, neg_hi, r[u], lo, hi);
            } else {
                UnitWords<32> rw;
                rw.r[0] = r[u * T::BPU]; rw.r[1] = r[u * T::BPU + T::BPU - 1];
                quantize_unit_bytes_fixed23<EO>(v, t.inv[u], t.cap23, neg_lo, neg_hi, rw, lo, hi);
            }
            if (EO) store_unit_even_odd(lo, hi, t.lp + u * kThreads * UB);
            else store_unit<FMT>(lo, hi, t.lp + u * kThreads * UB, t.lp2 + u * kThreads * UB2);
            if (DEC) {
                // the sum over the workers: the bytes biased to 1 .. 255, bytes 0, 2 and bytes 1, 3 of a
                // word spread over the 16-bit lanes of a word each (8 * 255 fits a lane)
                const uint32_t bl = lo ^ 0x80808080u, bh = hi ^ 0x80808080u;
                t.sum[u][0] += __byte_perm(bl, 0u, 0x4240); t.sum[u][1] += __byte_perm(bl, 0u, 0x4341);
                t.sum[u][2] += __byte_perm(bh, 0u, 0x4240); t.sum[u][3] += __byte_perm(bh, 0u, 0x4341);
            }
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

// Select mode: copies of the tile's rows of workers m0 .. m0 + cnt - 1 into shared memory, laid out
// [worker][unit][16 bytes][thread] so that every thread reads back only what it copied (no barrier).
// CNT > 0: cnt is that compile-time value (no predicates); CNT == 0: cnt at run time.
template <int CNT, int DT, int RNG>
__device__ __forceinline__ void stage_rows(uint4 *stage, const char *gp, size_t grow, int cnt)
{
    using E = Elem<DT>;
    constexpr int U = EncodeShape<DT, RNG>::UNITS, H = 8 / E::G;
    const int tid = threadIdx.x;
#pragma unroll
    for (int m = 0; m < kWorkerGroup; ++m) {
        if (CNT > 0 ? m < CNT : m < cnt) {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int h = 0; h < H; ++h)
                    copy_async16(stage + ((m * U + u) * H + h) * kThreads + tid, gp + (u * kThreads * 8 + h * E::G) * E::BYTES);
            gp += grow;
        }
    }
}

// Select mode: the largest magnitude over the staged workers of the 8 coordinates of unit u, as
// binary32 bit patterns.  bf16: two coordinates per word.  Its sign-magnitude halves read as
// signed 16-bit integers order the positive values, read as unsigned ones the negative values
// (sign bit set) above all others, so max |x| = max(smax & 0x7FFF, umax & 0x7FFF): two packed
// three-input maxima per two workers and word, no mask per element.  binary32: three-input
// maxima of absolute values, as the selector's kernel takes them (a NaN is skipped).
template <int CNT, int DT, int RNG>
__device__ __forceinline__ void staged_max_magnitude(const uint4 *stage, int u, int cnt, uint32_t (&amag)[8])
{
    using E = Elem<DT>;
    constexpr int U = EncodeShape<DT, RNG>::UNITS, H = 8 / E::G;
    const int tid = threadIdx.x;
    if (DT == UQ_F32) {
        float a[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int m = 0; m < kWorkerGroup; ++m) {
            if (CNT > 0 ? m < CNT : m < cnt) {
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const uint4 x = stage[((m * U + u) * H + h) * kThreads + tid];
                    a[4 * h + 0] = fmaxf(a[4 * h + 0], fabsf(__uint_as_float(x.x)));
                    a[4 * h + 1] = fmaxf(a[4 * h + 1], fabsf(__uint_as_float(x.y)));
                    a[4 * h + 2] = fmaxf(a[4 * h + 2], fabsf(__uint_as_float(x.z)));
                    a[4 * h + 3] = fmaxf(a[4 * h + 3], fabsf(__uint_as_float(x.w)));
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) amag[e] = __float_as_uint(a[e]);
    } else {
        uint32_t smax[4] = {0x80008000u, 0x80008000u, 0x80008000u, 0x80008000u}, umax[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int m = 0; m < kWorkerGroup; ++m) {
            if (CNT > 0 ? m < CNT : m < cnt) {
                const uint4 x = stage[(m * U + u) * kThreads + tid];
                const uint32_t w4[4] = { x.x, x.y, x.z, x.w };
#pragma unroll
                for (int c = 0; c < 4; ++c) { smax[c] = __vmaxs2(smax[c], w4[c]); umax[c] = __vmaxu2(umax[c], w4[c]); }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t am = __vmaxu2(smax[c] & 0x7FFF7FFFu, umax[c] & 0x7FFF7FFFu);
            amag[2 * c] = am << 16; amag[2 * c + 1] = am & 0xFFFF0000u;
        }
    }
}

// SEL: the kernel also finds and stores the shared scale indices (multi-scale, all M <= kWorkerGroup
// workers in one CTA): the tile's rows are copied to shared memory once (every thread its own
// units, so no barrier), read there for the maximum over the workers and again for quantization.
// DEC: decode mode (see the head of this file; int8 levels, 16-bit draws, one CTA per tile; with or without SEL).
template <int DT, int FMT, int RNG, int IDXB, bool SEL, bool DEC>
__global__ void __launch_bounds__(kThreads, (SEL ? 3 : DEC ? EncodeShape<DT, RNG>::MIN_CTAS_DEC : EncodeShape<DT, RNG>::MIN_CTAS))
encode_kernel(const __grid_constant__ EncodeParams p)
{
    static_assert(!DEC || (FMT == UQ_FMT_I8 && RNG == 16), "decode mode: int8 levels, 16-bit draws");
    grid_dependency_prologue();
    using T = TileState<DT, FMT, RNG, IDXB, DEC>;
    using E = Elem<DT>;
    using S = EncodeShape<DT, RNG>;
    using LF = LevelFmt<FMT>;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int U = T::U, H = T::H, BPU = T::BPU;
    const int tid = threadIdx.x, lane = tid & 31;
    __shared__ int32_t sh_thr[MULTI ? kWarps * 2 * UQ_MAX_SCALES : 1];   // select mode, slow paths: threshold tables
    const uint32_t first_tile_block = DEC ? p.row_blocks : 0u;
    if (DEC ? blockIdx.x < p.row_blocks : blockIdx.x >= p.main_blocks) {
        // A CTA of the second kind: each warp takes one segment boundary of one worker and, if the
        // boundary lies strictly inside a 256-coordinate row of a full tile, quantizes that row with
        // per-coordinate scales (the tile's own CTA skips it).  Keeping these rows out of the tile
        // CTAs keeps their lifetime short: the slow path no longer holds a whole CTA slot.
        // (decode mode: one warp takes the row of every worker, one after the other, and then decodes it)
        const uint32_t x = DEC ? blockIdx.x : blockIdx.x - p.main_blocks;
        const int m = DEC ? 0 : (int)(x % (uint32_t)p.v.M);
        const int64_t k = 1 + (int64_t)(DEC ? x : x / (uint32_t)p.v.M) * kWarps + (tid >> 5);
        if (k >= p.v.nseg) return;
        const int64_t b = __ldg(p.v.seg_off + k), prev = __ldg(p.v.seg_off + k - 1);
        const int64_t r0 = b & ~(int64_t)255;
        const int64_t full_end = p.v.d / S::TILE * S::TILE;          // rows beyond belong to the ragged tile's CTA
        if (b <= 0 || b == r0 || r0 >= full_end) return;           // not strictly inside a row of a full tile
        if (prev > r0 && prev <= b) return;                        // an earlier boundary in the same row takes it
        if (DEC) {
            // (select mode: the tile's own CTA stores the row's shared indices; this warp finds them for itself)
            const bool own = MULTI && p.select;
            int32_t *thr = sh_thr + (MULTI ? (tid >> 5) * 2 * UQ_MAX_SCALES : 0);
            for (int mm = 0; mm < p.v.M; ++mm) encode_span_general<DT, FMT, RNG, IDXB>(p, mm, r0, r0 + 256, lane, 32, own, thr);
            uint64_t kbits = 0;
            if (own) kbits = (uint64_t)select_unit<DT, IB, 4>(p.v, r0 + lane * 8, r0, thr);
            decode_unit_general<IDXB>(p, r0 + lane * 8, kbits, own);
            return;
        }
        encode_span_general<DT, FMT, RNG, IDXB>(p, m, r0, r0 + 256, lane, 32, MULTI && p.select,
                                                sh_thr + (MULTI ? (tid >> 5) * 2 * UQ_MAX_SCALES : 0));
        return;
    }
    // CTAs walk the tiles back to front (see launch_encode); a tile's CTAs take 8 workers each
    const uint32_t rev = p.main_blocks - 1u - (blockIdx.x - first_tile_block);
    const int64_t tile = (int64_t)(rev / p.groups);
    const int m0 = (int)(rev % p.groups) * kWorkerGroup;
    const int cnt = min(kWorkerGroup, p.v.M - m0);
    const int64_t t0 = tile * S::TILE;
    const int64_t t1 = min(t0 + (int64_t)S::TILE, p.v.d);

    // Philox block of the tile's first unit.  The units of a tile add less than 2^12 to it; the
    // straight-line path keeps the high word fixed (the per-worker table of the launch was made for
    // one high word), so a tile in which the low word wraps or whose high word is another one
    // (one launch in 2^35 coordinates) takes the general path like the ragged last tile.
    constexpr int BSH = RNG == 32 ? 2 : 3;                       // coordinates per Philox block, log2
    const uint64_t blk0 = (uint64_t)(p.coord0 >> BSH) + (uint64_t)tile * (uint32_t)(S::TILE >> BSH);
    const bool other_hi = (uint32_t)blk0 > 0xFFFFFFFFu - (uint32_t)(S::TILE >> BSH) || (uint32_t)(blk0 >> 32) != p.blk_hi;
    if (t1 - t0 != S::TILE || other_hi) {
        encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, -1, m0, m0 + cnt, sh_thr);
        if (DEC) decode_tile_slow<DT, RNG, IDXB>(p, t0, t1, false);
        return;
    }
    // every warp looks the segment up for itself (no shared memory, no barrier)
    const int j = warp_find_segment(p.v.seg_off, p.v.nseg, t0);
    if (segment_end(p.v.seg_off, p.v.nseg, j, p.v.d) < t1) {
        // A segment boundary crosses the tile (at most nseg - 1 tiles): a compact loop over the
        // rows of every worker, kept out of line so that its registers do not weigh on the path below.
        encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, j, m0, m0 + cnt, sh_thr);
        if (DEC) decode_tile_slow<DT, RNG, IDXB>(p, t0, t1, true);
        return;
    }
    T t;
    t.grow = (size_t)p.v.stride * E::BYTES;
    t.lrow = LF::row_bytes(p.v.stride);
    t.gp = (const char *)p.v.g + (size_t)m0 * t.grow + ((size_t)t0 + (size_t)tid * 8) * E::BYTES;
    uint4 q[U][H];
    typename IdxBits<IB>::T kbits[U];
    extern __shared__ uint4 stage[];                             // SEL: [worker][unit][16 bytes][thread]
    if (SEL) {
        t.sp = stage + tid;
        if (cnt == kWorkerGroup) stage_rows<kWorkerGroup, DT, RNG>(stage, t.gp, t.grow, cnt);
        else stage_rows<0, DT, RNG>(stage, t.gp, t.grow, cnt);
    } else {
        // the first worker's row and the shared indices are on their way during the set-up below
        load_units<false>(t, q);
        if (MULTI) {
            const uint8_t *ip = p.idx + ((size_t)t0 + (size_t)tid * 8) * IB / 8;
#pragma unroll
            for (int u = 0; u < U; ++u) kbits[u] = IdxBits<IB>::load(ip + u * kThreads * IB);
        }
    }
    // lane k holds s_k / W_j (single-scale: every lane holds s / W_j)
    constexpr int KMASK = IB < 4 ? (1 << IB) - 1 : UQ_MAX_SCALES - 1;    // lane L holds scale L & KMASK
    const float W = __ldg(p.v.W + j);
    float inv_lane = inv_scale(p.v.scales.s[lane & KMASK], W);
    if (lane < p.v.scales.N && not_finite(inv_lane) && p.status) atomicOr(p.status, (uint32_t)UQ_STATUS_SCALE_OVERFLOW);
    // a W so large (16-bit draws) or so small (32-bit) that the rescaled factors of the fast forms
    // would leave the normal range: the plain arithmetic
    if (RNG == 16 ? !sat_form_exact(inv_scale(p.v.scales.s[0], W))
                  : !fixed_form_exact(inv_scale(p.v.scales.s[p.v.scales.N - 1], W))) {
        if (SEL) copy_async_wait();
        encode_tile_slow<DT, FMT, RNG, IDXB>(p, t0, t1, -1, m0, m0 + cnt, sh_thr);
        if (DEC) decode_tile_slow<DT, RNG, IDXB>(p, t0, t1, false);
        return;
    }
    if (SEL) {
        // Scale selection and sharing for the tile (Algorithm 2 lines "Compute coordinate scales" and
        // "Scale sharing"): the largest magnitude over the workers decides the shared index (see
        // uq_select.cuh), found by bisection over the pass thresholds that lanes 0 .. N-1 hold.
        const int N = p.v.scales.N;
        const int32_t thr = lane < N ? pass_threshold(inv_lane, p.v.s_hat) : -1;
        const int top = N > 1 ? 1 << (31 - __clz(N - 1)) : 0;               // first step of the bisection
        const int32_t thr_top = __shfl_sync(0xFFFFFFFFu, thr, top);
        copy_async_wait();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t amag[8];
            if (cnt == kWorkerGroup) staged_max_magnitude<kWorkerGroup, DT, RNG>(stage, u, cnt, amag);
            else staged_max_magnitude<0, DT, RNG>(stage, u, cnt, amag);
            int k[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) k[e] = (top != 0 && (int32_t)amag[e] <= thr_top) ? top : 0;   // the first step
#pragma unroll 1
            for (int step = top >> 1; step >= 1; step >>= 1) {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if ((int32_t)amag[e] <= __shfl_sync(0xFFFFFFFFu, thr, k[e] + step)) k[e] += step;
            }
            typename IdxBits<IB>::T packed = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) packed |= (typename IdxBits<IB>::T)k[e] << (e * IB);
            kbits[u] = packed;
            store_unit_indices<IB>(p.idx, t0 + (int64_t)(u * kThreads + tid) * 8, packed);
        }
        load_units<true>(t, q);
    }
    if (RNG == 16) {
        inv_lane = __fmul_rn(inv_lane, 0.00390625f);
        t.sc = sat_constants(p.v.s_hat);
    } else {
        inv_lane = __fmul_rn(inv_lane, 8388608.0f);
        t.cap23 = __fmul_rn(p.v.s_hat, 8388608.0f);
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
    t.lp2 = lrow0 + LF::off2(t0, p.v.stride) + tid * (FMT == UQ_FMT_I6P ? 2 : 0);

    // decode mode: lane k holds the reconstruction factor of scale k, the sums start at zero
    float c_lane = 0.0f;
    if (DEC) {
        c_lane = decode_factor(W, p.v.scales.s[lane & KMASK], p.v.M);
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int k = 0; k < 4; ++k) t.sum[u][k] = 0u;
    }

    // The workers of the group straight-line, with no loop around them: all 8, or (the last group
    // of a job whose M is not a multiple of 8) 4, 2 and 1 of them as the count's bits say.
    if (cnt == kWorkerGroup) {
        encode_workers<kWorkerGroup, false, SEL>(p, t, m0, q);
    } else {
        int m = m0;
        if (cnt & 4) {
            if (cnt & 3) encode_workers<4, true, SEL>(p, t, m, q);
            else encode_workers<4, false, SEL>(p, t, m, q);
            m += 4;
        }
        if (cnt & 2) {
            if (cnt & 1) encode_workers<2, true, SEL>(p, t, m, q);
            else encode_workers<2, false, SEL>(p, t, m, q);
            m += 2;
        }
        if (cnt & 1) encode_workers<1, false, SEL>(p, t, m, q);
    }
    if (DEC) {
        // Algorithm 1 / 2, lines "AllReduce gradients" and "Reconstruct gradient" for the tile: the sum
        // of a coordinate leaves its lane, loses the bias, and is multiplied by the factor of the
        // coordinate's scale (the same three operations as the aggregation kernel's)
        const int bias = 128 * p.v.M;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t r[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t lanes = t.sum[DEC ? u : 0][(e >> 2) * 2 + (e & 1)];
                const int sum = (int)((lanes >> (16 * ((e & 3) >> 1))) & 0xFFFFu) - bias;
                const float c = MULTI ? __shfl_sync(0xFFFFFFFFu, c_lane, (int)(uint32_t)(kbits[u] >> (e * IB))) : c_lane;
                r[e] = __float_as_uint(__fmul_rn((float)sum, c));
            }
            st_stream256(p.out + t0 + (int64_t)(u * kThreads + tid) * 8, r);
        }
    }
}

template <int DT, int FMT, int RNG, int IDXB, bool SEL = false, bool DEC = false>
static cudaError_t launch(EncodeParams p, cudaStream_t st)
{
    using S = EncodeShape<DT, RNG>;
    const int64_t ntiles = (p.v.d + S::TILE - 1) / S::TILE;
    p.reserved = 0u;
    p.groups = (uint32_t)((p.v.M + kWorkerGroup - 1) / kWorkerGroup);
    int64_t blocks = ntiles * p.groups;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    p.main_blocks = (uint32_t)blocks;
    int64_t rows = 0;
    if (p.v.seg_off != nullptr && p.v.nseg > 1) rows = (int64_t)((p.v.nseg - 1 + kWarps - 1) / kWarps) * (DEC ? 1 : p.v.M);
    blocks += rows;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    p.row_blocks = (uint32_t)rows;
    constexpr int BSH = RNG == 32 ? 2 : 3;
    p.blk_hi = (uint32_t)((uint64_t)(p.coord0 >> BSH) >> 32);
    for (int m = 0; m < UQ_MAX_WORKERS; ++m)
        p.wpart[m] = philox_worker_part(p.key, p.blk_hi, (uint32_t)(p.worker0 + (m < p.v.M ? m : 0)));
    if (SEL) {
        // the copies of the tile's rows: up to kWorkerGroup workers * TILE coordinates (64 KiB)
        const size_t smem = (size_t)(p.v.M < kWorkerGroup ? p.v.M : kWorkerGroup) * S::TILE * Elem<DT>::BYTES;
        // more than 48 KiB of dynamic shared memory needs an opt-in per kernel and device (the call
        // is idempotent, so a race between host threads on the flag is harmless)
        static bool opted_in[64] = {};
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64 || !opted_in[dev]) {
            e = cudaFuncSetAttribute(encode_kernel<DT, FMT, RNG, IDXB, SEL, DEC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kWorkerGroup * S::TILE * Elem<DT>::BYTES);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) opted_in[dev] = true;
        }
        launch_k_smem(encode_kernel<DT, FMT, RNG, IDXB, SEL, DEC>, (unsigned)blocks, kThreads, smem, st, p);
    } else {
        launch_k(encode_kernel<DT, FMT, RNG, IDXB, SEL, DEC>, (unsigned)blocks, kThreads, st, p);
    }
    return cudaGetLastError();
}

template <int DT, int FMT, int RNG>
static cudaError_t dispatch_idx(const EncodeParams &p, int idx_bits, cudaStream_t st)
{
    if constexpr (FMT == UQ_FMT_I8 && RNG == 16) {
        if (p.out != nullptr && !p.select) {          // decode mode (the caller has checked M <= kWorkerGroup)
            switch (idx_bits) {
            case 0: return launch<DT, FMT, RNG, 0, false, true>(p, st);
            case 1: return launch<DT, FMT, RNG, 1, false, true>(p, st);
            case 2: return launch<DT, FMT, RNG, 2, false, true>(p, st);
            case 4: return launch<DT, FMT, RNG, 4, false, true>(p, st);
            default: return launch<DT, FMT, RNG, 8, false, true>(p, st);
            }
        }
    }
    if constexpr (FMT == UQ_FMT_I8 && RNG == 16) {
        if (p.out != nullptr && p.select) {           // select mode and decode mode together
            switch (idx_bits) {
            case 1: return launch<DT, FMT, RNG, 1, true, true>(p, st);
            case 2: return launch<DT, FMT, RNG, 2, true, true>(p, st);
            case 4: return launch<DT, FMT, RNG, 4, true, true>(p, st);
            default: return launch<DT, FMT, RNG, 8, true, true>(p, st);
            }
        }
    }
    if (p.select) {
        switch (idx_bits) {
        case 1: return launch<DT, FMT, RNG, 1, true>(p, st);
        case 2: return launch<DT, FMT, RNG, 2, true>(p, st);
        case 4: return launch<DT, FMT, RNG, 4, true>(p, st);
        default: return launch<DT, FMT, RNG, 8, true>(p, st);
        }
    }
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
