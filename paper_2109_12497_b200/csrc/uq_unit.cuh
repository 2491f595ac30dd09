// One unit of the encoders: eight consecutive coordinates of one worker turned into levels.
// Shared by the streaming encoder (one worker per CTA) and the fused select + encode kernel
// (all workers per thread).
#pragma once
#include "uq_device.cuh"

namespace uq {

// (float)s_k / W with one IEEE division; 0 for an all-zero segment.
__device__ __forceinline__ float inv_scale(int32_t s, float W)
{
    return W > 0.0f ? __fdiv_rn((float)s, W) : 0.0f;
}

__device__ __forceinline__ bool not_finite(float x) { return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u; }

// The idx_bits * 8 bits that belong to 8 consecutive coordinates starting at a multiple of 8.
template <int IDXB> struct IdxBits;
// load: indices written by an earlier kernel; load_written: indices that this kernel wrote itself
// (the read-only path must not be used for them).
template <> struct IdxBits<1> {
    using T = uint32_t;
    static __device__ __forceinline__ T load(const uint8_t *p) { return __ldg(p); }
    static __device__ __forceinline__ T load_written(const uint8_t *p) { return __ldcg(p); }
};
template <> struct IdxBits<2> {
    using T = uint32_t;
    static __device__ __forceinline__ T load(const uint8_t *p) { return __ldg((const uint16_t *)p); }
    static __device__ __forceinline__ T load_written(const uint8_t *p) { return __ldcg((const uint16_t *)p); }
};
template <> struct IdxBits<4> {
    using T = uint32_t;
    static __device__ __forceinline__ T load(const uint8_t *p) { return __ldg((const uint32_t *)p); }
    static __device__ __forceinline__ T load_written(const uint8_t *p) { return __ldcg((const uint32_t *)p); }
};
template <> struct IdxBits<8> {
    using T = uint64_t;
    static __device__ __forceinline__ T load(const uint8_t *p) { return __ldg((const unsigned long long *)p); }
    static __device__ __forceinline__ T load_written(const uint8_t *p) { return __ldcg((const unsigned long long *)p); }
};

// Eight coordinates: magnitudes scaled by inv[e], random words from the block(s) starting at
// (blk_lo, blk_hi), levels gathered four to a word, signs applied bytewise (`neg` holds 0xFF in
// the bytes of negative coordinates), packed into the wire format and stored at `dst`.
// coordinate c uses word c%4 of block c/4 (32-bit draws) or half (c%8)%2 of word (c%8)/2 of block
// c/8 (16-bit draws).
// The random words of a unit: RNG == 32 takes blocks blk_lo and blk_lo + 1 (blk_lo is even: no
// carry), RNG == 16 the single block blk_lo.
template <int RNG> struct UnitWords { uint4 r[RNG == 32 ? 2 : 1]; };

template <int RNG>
__device__ __forceinline__ UnitWords<RNG> unit_words(const PhiloxKey &key, uint32_t blk_lo, uint32_t blk_hi, uint32_t m)
{
    UnitWords<RNG> w;
    if (RNG == 32) {
        const uint32_t b[2] = { blk_lo, blk_lo + 1u };
        uint4 r[2];
        philox4x32_10_xN<2>(key, b, blk_hi, m, r);
        w.r[0] = r[0]; w.r[RNG == 32 ? 1 : 0] = r[1];
    } else {
        w.r[0] = philox4x32_10(key, blk_lo, blk_hi, m);
    }
    return w;
}

// The signed levels of a unit as bytes: coordinates 0..3 in `lo`, 4..7 in `hi`.
template <int RNG>
__device__ __forceinline__ void quantize_unit_bytes(const float (&v)[8], const float (&inv)[8], float cap,
                                                    uint32_t neg_lo, uint32_t neg_hi, const UnitWords<RNG> &rw,
                                                    uint32_t &lo, uint32_t &hi)
{
    constexpr uint32_t LB = RNG == 32 ? kLevelByte23 : kLevelByte16;
    uint32_t z[8];
    if (RNG == 32) {
        const uint4 r0 = rw.r[0], r1 = rw.r[RNG == 32 ? 1 : 0];
        const uint32_t w[8] = { r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w };
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = level_draw23(scaled_magnitude(v[e], inv[e], cap), w[e]);
    } else {
        const uint4 r = rw.r[0];
        const uint32_t w[4] = { r.x, r.y, r.z, r.w };
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t h = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
            z[e] = level_draw16(scaled_magnitude(v[e], inv[e], cap), h);
        }
    }
    lo = negate_bytes(gather_bytes<LB>(z[0], z[1], z[2], z[3]), neg_lo);
    hi = negate_bytes(gather_bytes<LB>(z[4], z[5], z[6], z[7]), neg_hi);
}

// The same for 23-bit draws in the fixed-point form (level_draw23_fixed): inv23[e] = inv[e] * 2^23,
// cap23 = cap * 2^23.  fixed_form_exact says whether a tile may take it, given the largest of its
// factors: beyond 2^100 (W below 2^-93 or so; also Inf and NaN) the scaled factor could overflow,
// and the tile takes the plain arithmetic.
__device__ __forceinline__ bool fixed_form_exact(float inv_max) { return inv_max <= 1.2676506e30f; }

// EO (here and below): `lo` takes the even coordinates 0, 2, 4, 6 and `hi` the odd ones, with the
// sign masks in the same order (unit_signs<DT, true>); the 4-bit store merges such a pair without
// a permute (store_unit_even_odd).
template <bool EO = false>
__device__ __forceinline__ void quantize_unit_bytes_fixed23(const float (&v)[8], const float (&inv23)[8], float cap23,
                                                            uint32_t neg_lo, uint32_t neg_hi, const UnitWords<32> &rw,
                                                            uint32_t &lo, uint32_t &hi)
{
    const uint4 r0 = rw.r[0], r1 = rw.r[1];
    const uint32_t w[8] = { r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w };
    uint32_t z[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) z[e] = level_draw23_fixed(v[e], inv23[e], cap23, w[e]);
    constexpr int S = EO ? 2 : 1, B = EO ? 1 : 4;               // coordinate step within a word, first of `hi`
    lo = negated_bytes_to_signed(gather_bytes<kLevelByte23Fixed>(z[0], z[S], z[2 * S], z[3 * S]), neg_lo);
    hi = negated_bytes_to_signed(gather_bytes<kLevelByte23Fixed>(z[B], z[B + S], z[B + 2 * S], z[B + 3 * S]), neg_hi);
}

// The same for 16-bit draws with the clamp in saturating arithmetic (level_draw16_sat): inv256[e]
// is the coordinate's factor divided by 256, (c0, adj) come from sat_constants(cap).
struct SatConstants { float c0; uint32_t adj; };
__device__ __forceinline__ SatConstants sat_constants(float cap)
{
    SatConstants c;
    c.c0 = __fsub_rn(1.0f, __fmul_rn(cap, 0.00390625f));
    c.adj = 0xFFFFFFFFu - ((127u - (uint32_t)cap) << 16);
    return c;
}
// Whether the saturating form may be used with smallest factor inv0 (= scales[0] / W): dividing a
// factor below 2^-100 by 256 could round.  (0, Inf and NaN divide exactly.)
__device__ __forceinline__ bool sat_form_exact(float inv0) { return !(inv0 > 0.0f && inv0 < 7.888609052e-31f); }

template <bool EO = false>
__device__ __forceinline__ void quantize_unit_bytes_sat16(const float (&v)[8], const float (&inv256)[8], const SatConstants &sc,
                                                          uint32_t neg_lo, uint32_t neg_hi, const uint4 &r, uint32_t &lo,
                                                          uint32_t &hi)
{
    const uint32_t w[4] = { r.x, r.y, r.z, r.w };
    uint32_t z[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const uint32_t h = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
        z[e] = level_draw16_sat(v[e], inv256[e], sc.c0, sc.adj, h);
    }
    constexpr int S = EO ? 2 : 1, B = EO ? 1 : 4;
    lo = negate_bytes(gather_bytes<2>(z[0], z[S], z[2 * S], z[3 * S]), neg_lo);
    hi = negate_bytes(gather_bytes<2>(z[B], z[B + S], z[B + 2 * S], z[B + 3 * S]), neg_hi);
}

// The level bytes of a unit packed into the wire format and stored.
template <int FMT> __device__ __forceinline__ void store_unit(uint32_t lo, uint32_t hi, void *dst, void *dst2)
{
    // plain stores (not evict-first ones): the aggregation kernel that follows reads the levels
    // back, and what is still in L2 then costs no DRAM read (measured: 7-9 % off that kernel)
    if (FMT == UQ_FMT_I8) *(uint2 *)dst = make_uint2(lo, hi);
    else if (FMT == UQ_FMT_I4X2) *(uint32_t *)dst = bytes_to_nibbles(lo, hi);
    else if (FMT == UQ_FMT_I2X4) *(unsigned short *)dst = (unsigned short)bytes_to_crumbs(lo, hi);
    else {                                          // 6-bit: bits 0..3 as nibbles, bits 4..5 as 2-bit fields
        *(uint32_t *)dst = bytes_to_nibbles(lo, hi);
        *(unsigned short *)dst2 = (unsigned short)bytes_to_crumbs(lo >> 4, hi >> 4);
    }
}

// 4-bit levels from a unit in even / odd order: byte k of `even` is coordinate 2k and becomes the
// low nibble of byte k, byte k of `odd` the high one.
__device__ __forceinline__ void store_unit_even_odd(uint32_t even, uint32_t odd, void *dst)
{
    *(uint32_t *)dst = (even & 0x0F0F0F0Fu) | ((odd << 4) & 0xF0F0F0F0u);
}

template <int FMT, int RNG>
__device__ __forceinline__ void quantize_unit_words(const float (&v)[8], const float (&inv)[8], float cap,
                                                    uint32_t neg_lo, uint32_t neg_hi, const UnitWords<RNG> &rw,
                                                    void *dst, void *dst2, bool store = true)
{
    uint32_t lo, hi;
    quantize_unit_bytes<RNG>(v, inv, cap, neg_lo, neg_hi, rw, lo, hi);
    if (store) store_unit<FMT>(lo, hi, dst, dst2);
}

template <int FMT, int RNG>
__device__ __forceinline__ void quantize_unit(const float (&v)[8], const float (&inv)[8], float cap,
                                              uint32_t neg_lo, uint32_t neg_hi, const PhiloxKey &key,
                                              uint32_t blk_lo, uint32_t blk_hi, uint32_t m, void *dst,
                                              void *dst2, bool store = true)
{
    quantize_unit_words<FMT, RNG>(v, inv, cap, neg_lo, neg_hi, unit_words<RNG>(key, blk_lo, blk_hi, m), dst, dst2, store);
}

// The sign masks of a unit, from the raw loaded words (before any padding is zeroed).
template <int DT, bool EO = false> __device__ __forceinline__ void unit_signs(const uint4 *q, uint32_t &neg_lo, uint32_t &neg_hi)
{
    static_assert(!EO || DT == UQ_F32, "even / odd order: binary32 only (for bf16 the masks would cost two more permutes)");
    if (EO) {
        neg_lo = sign_bytes_f32(__uint_as_float(q[0].x), __uint_as_float(q[0].z), __uint_as_float(q[1].x),
                                __uint_as_float(q[1].z));
        neg_hi = sign_bytes_f32(__uint_as_float(q[0].y), __uint_as_float(q[0].w), __uint_as_float(q[1].y),
                                __uint_as_float(q[1].w));
    } else if (DT == UQ_F32) {
        neg_lo = sign_bytes_f32(__uint_as_float(q[0].x), __uint_as_float(q[0].y), __uint_as_float(q[0].z),
                                __uint_as_float(q[0].w));
        neg_hi = sign_bytes_f32(__uint_as_float(q[1].x), __uint_as_float(q[1].y), __uint_as_float(q[1].z),
                                __uint_as_float(q[1].w));
    } else {
        neg_lo = sign_bytes_bf16(q[0].x, q[0].y);
        neg_hi = sign_bytes_bf16(q[0].z, q[0].w);
    }
}

}  // namespace uq
