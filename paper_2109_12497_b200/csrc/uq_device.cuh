// Device-side helpers shared by the uq kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "uq.h"

namespace uq {

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch: every kernel of the library is launched with the attribute that
// lets the GPU schedule its CTAs while the kernel before it in the stream is still draining, and
// starts with grid_dependency_prologue(): it first lets the kernel AFTER it be scheduled the same
// way, then waits until the kernel before it has completed and its writes are visible.  No read of
// global memory may come before the prologue.  What overlaps is launch latency and the ramp of the
// CTAs, not the work; a predecessor that knows nothing of this (a framework kernel, a copy) simply
// counts as complete when it ends.  -DUQ_NO_PDL launches the plain way.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void grid_dependency_prologue()
{
#ifndef UQ_NO_PDL
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
}

template <typename... P, typename... A>
inline void launch_k_smem(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t st, A &&...args)
{
#ifdef UQ_NO_PDL
    kernel<<<grid, block, smem_bytes, st>>>(static_cast<A &&>(args)...);
#else
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<A &&>(args)...);    // an error stays for cudaGetLastError()
#endif
}

template <typename... P, typename... A>
inline void launch_k(void (*kernel)(P...), dim3 grid, dim3 block, cudaStream_t st, A &&...args)
{
    launch_k_smem(kernel, grid, block, 0, st, static_cast<A &&>(args)...);
}

constexpr int kThreads = 256;            // threads per CTA in every streaming kernel
constexpr int kWarps = kThreads / 32;
constexpr int kNormTile = 8192;          // coordinates per partial of the norm reduction

struct ScaleSet {                        // the scale set s_ of the multi-scale quantizer
    int32_t s[UQ_MAX_SCALES];
    int32_t N;
};

// The low two bits of the eight bytes of (lo, hi), coordinate order kept: byte t of lo lands in
// bits 2t..2t+1, byte t of hi in bits 8+2t..9+2t (levels -1, 0, 1 as two's-complement 2-bit fields).
// One multiply gathers a word's four fields: with x = c0 + c1 2^8 + c2 2^16 + c3 2^24 (c < 4) and
// K = 2^24 + 2^18 + 2^12 + 2^6 the product has c0, c1, c2, c3 at bits 24, 26, 28, 30; every other
// partial product that stays below 2^32 lies at bit 22 or lower and their sum is below 2^24, so
// byte 3 of x * K is the packed byte.  Bits 16..31 of the result are unspecified.
__device__ __forceinline__ uint32_t bytes_to_crumbs(uint32_t lo, uint32_t hi)
{
    constexpr uint32_t K = (1u << 24) | (1u << 18) | (1u << 12) | (1u << 6);
    return __byte_perm((lo & 0x03030303u) * K, (hi & 0x03030303u) * K, 0x4473);
}

// ---------------------------------------------------------------------------------------------
// loads / stores
// ---------------------------------------------------------------------------------------------

// Streaming 128-bit load: the data is read once, keep it out of L1.
__device__ __forceinline__ uint4 ld_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Streaming 64-bit load (8-byte aligned).
__device__ __forceinline__ uint2 ld_stream64(const void *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// The same loads on the coherent path (no .nc): for memory that another GPU wrote (a peer's rows
// read over NVLink), which must not be assumed read-only or served from a stale non-coherent line.
__device__ __forceinline__ uint4 ld_coherent(const void *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint2 ld_coherent64(const void *p)
{
    uint2 v;
    asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}

template <typename T> __device__ __forceinline__ void st_stream(T *p, T v) { __stcs(p, v); }

// 16 bytes from global memory straight into shared memory (no register in between); the copies of
// a thread are complete for that thread after copy_async_wait().
__device__ __forceinline__ void copy_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void copy_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// 256-bit streaming load / store (sm_100 and later): 32 bytes per lane in one instruction.
// The address must be 32-byte aligned.
struct alignas(32) uint8x { uint32_t w[8]; };

__device__ __forceinline__ uint8x ld_stream256(const void *p)
{
    uint8x v;
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                   "=r"(v.w[7])
                 : "l"(p));
    return v;
}

// 256-bit load / store of data that the same kernel both reads and writes (coherent path).
__device__ __forceinline__ void ld256(const void *p, float (&f)[8])
{
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(f[0]), "=f"(f[1]), "=f"(f[2]), "=f"(f[3]), "=f"(f[4]), "=f"(f[5]), "=f"(f[6]), "=f"(f[7])
                 : "l"(p) : "memory");
}

__device__ __forceinline__ void st256(void *p, const float (&f)[8])
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(f[4]), "f"(f[5]), "f"(f[6]), "f"(f[7])
                 : "memory");
}

__device__ __forceinline__ void st_stream256(void *p, const uint32_t (&w)[8])
{
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Coordinates per 16-byte granule, and unpacking of a granule to binary32.
template <int DT> struct Elem;
template <> struct Elem<UQ_F32> {
    static constexpr int G = 4;
    static constexpr int BYTES = 4;
    __device__ static __forceinline__ void unpack(const uint4 &q, float (&v)[4])
    {
        v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y);
        v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
    }
};
template <> struct Elem<UQ_BF16> {
    static constexpr int G = 8;
    static constexpr int BYTES = 2;
    __device__ static __forceinline__ void unpack(const uint4 &q, float (&v)[8])
    {
        v[0] = bf16lo(q.x); v[1] = bf16hi(q.x); v[2] = bf16lo(q.y); v[3] = bf16hi(q.y);
        v[4] = bf16lo(q.z); v[5] = bf16hi(q.z); v[6] = bf16lo(q.w); v[7] = bf16hi(q.w);
    }
};

// ---------------------------------------------------------------------------------------------
// segments
// ---------------------------------------------------------------------------------------------

// The segment that holds coordinate i: smallest j with seg_off[j+1] > i, clamped to
// [0, nseg-1] so that a malformed table can never index outside W.
__device__ __forceinline__ int find_segment(const int64_t *__restrict__ seg_off, int nseg, int64_t i)
{
    if (seg_off == nullptr) return 0;
    int lo = 0, hi = nseg - 1;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (__ldg(seg_off + mid + 1) <= i) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Advance j (a segment at or before coordinate i's) to the segment holding i.
__device__ __forceinline__ int advance_segment(const int64_t *__restrict__ seg_off, int nseg, int j, int64_t i)
{
    while (j + 1 < nseg && __ldg(seg_off + j + 1) <= i) ++j;
    return j;
}

__device__ __forceinline__ int64_t segment_end(const int64_t *__restrict__ seg_off, int nseg, int j, int64_t d)
{
    return (seg_off == nullptr || j + 1 >= nseg) ? d : __ldg(seg_off + j + 1);
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10, counter = (block low, block high, worker, tag), key = seed; the rounding draws use tag 0
// ---------------------------------------------------------------------------------------------

// The ten round keys (uniform over the grid).  8-byte aligned: inside kernel parameters the keys are
// fetched two at a time, and a table that starts on an odd word costs the encoders 6-9 % (measured).
struct alignas(8) PhiloxKey { uint32_t k0[10], k1[10]; };

__host__ __device__ __forceinline__ PhiloxKey philox_key(uint64_t seed)
{
    PhiloxKey k;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = a; k.k1[r] = b;
        a += 0x9E3779B9u; b += 0xBB67AE85u;
    }
    return k;
}

__device__ __forceinline__ uint4 philox4x32_10(const PhiloxKey &k, uint32_t block_lo, uint32_t block_hi, uint32_t worker,
                                               uint32_t tag = 0u)
{
    uint32_t c0 = block_lo, c1 = block_hi, c2 = worker, c3 = tag;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.k0[r];
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.k1[r];
        c1 = (uint32_t)p1; c3 = (uint32_t)p0; c0 = n0; c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// N blocks at once, block n at counter (block_lo[n], block_hi, worker): the N chains advance
// round by round together, so one fetch of a round key serves all of them and the chains' wide
// multiplies overlap.
template <int N>
__device__ __forceinline__ void philox4x32_10_xN(const PhiloxKey &k, const uint32_t (&block_lo)[N], uint32_t block_hi,
                                                 uint32_t worker, uint4 (&out)[N])
{
    uint32_t c0[N], c1[N], c2[N], c3[N];
#pragma unroll
    for (int n = 0; n < N; ++n) { c0[n] = block_lo[n]; c1[n] = block_hi; c2[n] = worker; c3[n] = 0u; }
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t k0 = k.k0[r], k1 = k.k1[r];
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const uint64_t p0 = (uint64_t)0xD2511F53u * c0[n];
            const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2[n];
            const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1[n] ^ k0;
            const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3[n] ^ k1;
            c1[n] = (uint32_t)p1; c3[n] = (uint32_t)p0; c0[n] = n0; c2[n] = n2;
        }
    }
#pragma unroll
    for (int n = 0; n < N; ++n) out[n] = make_uint4(c0[n], c1[n], c2[n], c3[n]);
}

// The same block number for N workers at once (worker[n] in counter word 2).
template <int N>
__device__ __forceinline__ void philox4x32_10_workers(const PhiloxKey &k, uint32_t block_lo, uint32_t block_hi,
                                                      const uint32_t (&worker)[N], uint4 (&out)[N])
{
    uint32_t c0[N], c1[N], c2[N], c3[N];
#pragma unroll
    for (int n = 0; n < N; ++n) { c0[n] = block_lo; c1[n] = block_hi; c2[n] = worker[n]; c3[n] = 0u; }
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t k0 = k.k0[r], k1 = k.k1[r];
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const uint64_t p0 = (uint64_t)0xD2511F53u * c0[n];
            const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2[n];
            const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1[n] ^ k0;
            const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3[n] ^ k1;
            c1[n] = (uint32_t)p1; c3[n] = (uint32_t)p0; c0[n] = n0; c2[n] = n2;
        }
    }
#pragma unroll
    for (int n = 0; n < N; ++n) out[n] = make_uint4(c0[n], c1[n], c2[n], c3[n]);
}

// The first two rounds of a block split by what they depend on.  Of the counter
// (block low, block high, worker, 0) only word 0 differs between the threads of a tile and only
// word 2 between the workers, and the two do not meet before the second round:
//   round 0: c0 = hi(M1*worker) ^ block_high ^ k0[0]   c1 = lo(M1*worker)       (per worker)
//            c2 = hi(M0*block_low) ^ k1[0]             c3 = lo(M0*block_low)    (per block)
//   round 1: c0 = hi(M1*c2) ^ c1 ^ k0[1]   c1 = lo(M1*c2)   c2 = hi(M0*c0) ^ c3 ^ k1[1]   c3 = lo(M0*c0)
// so a thread that draws the same block for several workers keeps {hi, lo}(M1*c2) and c3 of round 0
// (PhiloxBlockPart), takes the per-worker words from a table made once per launch
// (PhiloxWorkerPart, uniform over the grid), joins them with two three-input XORs and runs the
// remaining eight rounds: 34 instead of 40 multiply / XOR instructions per block.
struct PhiloxBlockPart { uint32_t a, b, c3; };       // hi(M1*c2), lo(M1*c2), c3 after round 0
struct PhiloxWorkerPart { uint32_t u1, hq, lq; };    // c1 after round 0; hi, lo of M0 * (c0 after round 0)

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;

__device__ __forceinline__ PhiloxBlockPart philox_block_part(const PhiloxKey &k, uint32_t block_lo)
{
    PhiloxBlockPart r;
    const uint64_t p0 = (uint64_t)kPhiloxM0 * block_lo;
    r.c3 = (uint32_t)p0;
    const uint64_t p1 = (uint64_t)kPhiloxM1 * ((uint32_t)(p0 >> 32) ^ k.k1[0]);
    r.a = (uint32_t)(p1 >> 32); r.b = (uint32_t)p1;
    return r;
}

__host__ __device__ __forceinline__ PhiloxWorkerPart philox_worker_part(const PhiloxKey &k, uint32_t block_hi, uint32_t worker)
{
    PhiloxWorkerPart w;
    const uint64_t pw = (uint64_t)kPhiloxM1 * worker;
    w.u1 = (uint32_t)pw;
    const uint64_t q0 = (uint64_t)kPhiloxM0 * ((uint32_t)(pw >> 32) ^ block_hi ^ k.k0[0]);
    w.hq = (uint32_t)(q0 >> 32); w.lq = (uint32_t)q0;
    return w;
}

// Rounds 1 (the joining XORs) to 9 of N blocks of one worker, advanced together.
template <int N>
__device__ __forceinline__ void philox_join(const PhiloxKey &k, const PhiloxBlockPart (&blk)[N], const PhiloxWorkerPart &w,
                                            uint4 (&out)[N])
{
    uint32_t c0[N], c1[N], c2[N], c3[N];
#pragma unroll
    for (int n = 0; n < N; ++n) {
        c0[n] = blk[n].a ^ w.u1 ^ k.k0[1];
        c1[n] = blk[n].b;
        c2[n] = w.hq ^ blk[n].c3 ^ k.k1[1];
        c3[n] = w.lq;
    }
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        const uint32_t k0 = k.k0[r], k1 = k.k1[r];
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const uint64_t p0 = (uint64_t)kPhiloxM0 * c0[n];
            const uint64_t p1 = (uint64_t)kPhiloxM1 * c2[n];
            const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1[n] ^ k0;
            const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3[n] ^ k1;
            c1[n] = (uint32_t)p1; c3[n] = (uint32_t)p0; c0[n] = n0; c2[n] = n2;
        }
    }
#pragma unroll
    for (int n = 0; n < N; ++n) out[n] = make_uint4(c0[n], c1[n], c2[n], c3[n]);
}

// ---------------------------------------------------------------------------------------------
// one coordinate of Q_s
// ---------------------------------------------------------------------------------------------

// x = min(|v| * inv, cap) with a single rounding; NaN collapses to cap.
__device__ __forceinline__ float scaled_magnitude(float v, float inv, float cap)
{
    return fminf(__fmul_rn(fabsf(v), inv), cap);
}

// 23-bit draw.  Returns a word whose LOW byte is the unsigned level
//   floor(x) + [h < rint((x - floor(x)) * 2^23)],  h = word >> 9,  0 <= x <= 127.
// t = x + 2^23 rounded down holds floor(x) in its low mantissa bits; t - (2^23 + 1) = floor(x) - 1
// exactly, so x - that is p + 1 with one rounding: its mantissa is rint(p * 2^23), and the carry
// into the exponent makes it 2^23 when p rounds up to 1.  The draw is placed under the same
// exponent by one funnel shift, so the test is a single unsigned compare.
__device__ __forceinline__ uint32_t level_draw23(float x, uint32_t word)
{
    const float t = __fadd_rd(x, 8388608.0f);
    const float p1 = __fsub_rn(x, __fsub_rn(t, 8388609.0f));
    const uint32_t hb = __funnelshift_r(word, 0x7Fu, 9);          // 0x3F800000 | (word >> 9)
    return __float_as_uint(t) + (hb < __float_as_uint(p1) ? 1u : 0u);
}
constexpr uint32_t kLevelByte23 = 0;      // which byte of the returned word holds the level

// The same level from the fixed-point form of x (the fast path of the encoder).  inv23 = inv * 2^23
// and cap23 = cap * 2^23, both exact, so |v| * inv23 = x * 2^23 with the rounding of x (the caller
// checks that inv23 is finite; a product below the normal range gives threshold 0 either way), and
//   T = rint(min(x, cap) * 2^23) = floor(x) * 2^23 + rint(p * 2^23)
// by one conversion (ties to even; x >= 1 is a multiple of 2^-23, so only p < 1 is rounded, and a
// p that rounds up to 1 carries into the level, as it must: then every draw rounds up).  With
// r = word >> 9 the level is L = (T + 2^23 - 1 - r) >> 23 = ceil((T - r) / 2^23), so
// -L = floor((r - T) / 2^23).  The function converts the negated product (-T, exactly) and returns
// y = 2 (-T) + (word >> 8) = 2 (r - T) + (0 or 1): byte 3 of y is -L as a two's-complement byte
// (-127 .. 0), the stray low bit changes no floor.  negated_bytes_to_signed puts the signs on.
__device__ __forceinline__ uint32_t level_draw23_fixed(float v, float inv23, float cap23, uint32_t word)
{
    const uint32_t Tn = (uint32_t)__float2int_rn(fmaxf(__fmul_rn(-fabsf(v), inv23), -cap23));
    return Tn + Tn + (word >> 8);
}
constexpr uint32_t kLevelByte23Fixed = 3;

// 16-bit draw.  Returns a word whose byte 2 is the unsigned level.
// x + 128 rounds x to 16 fractional bits (ties to even): the mantissa of the sum is
// floor(x) * 2^16 + rint(p * 2^16); adding 0xFFFF - h carries into bit 16 iff
// h < rint(p * 2^16) (one three-input add: the subtraction is an operand modifier).
__device__ __forceinline__ uint32_t level_draw16(float x, uint32_t h)
{
    return __float_as_uint(__fadd_rn(x, 128.0f)) + 0xFFFFu - h;
}
constexpr uint32_t kLevelByte16 = 2;

// The same level with the clamp folded into saturating arithmetic (both on the FMA pipe, where the
// min of the form above is an ALU instruction).  inv256 = inv / 256 exactly (the caller checks that
// inv is 0 or at least 2^-100, so nothing is lost to a subnormal), hence |v| * inv256 = x / 256
// with the rounding of x.  c0 = 1 - cap / 256: the saturating sum reaches 1.0 exactly where x
// reaches cap, and below 1.0 its unit in the last place is 2^-24, i.e. 2^-16 in x (ties to even as
// before, since c0 is an even multiple of it).  As an integer the sum is
//   0x3F000000 + (128 - cap) * 2^16 + floor(x) * 2^16 + rint(p * 2^16),
// and subtracting h + 1 borrows from the level field iff h >= rint(p * 2^16).  With
// adj = -1 - (127 - cap) * 2^16 byte 2 of the result is the level.  The saturating product turns a
// NaN (0 * Inf, a NaN input) into 0 and so into level 0; Inf saturates to level cap.
__device__ __forceinline__ float mul_sat(float a, float b)
{
    float d;
    asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ float add_sat(float a, float b)
{
    float d;
    asm("add.rn.sat.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ uint32_t level_draw16_sat(float v, float inv256, float c0, uint32_t adj, uint32_t h)
{
    return __float_as_uint(add_sat(mul_sat(fabsf(v), inv256), c0)) - h + adj;
}

// Gathers byte B of four words into one word (coordinate order = byte order).
template <uint32_t B> __device__ __forceinline__ uint32_t gather_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    constexpr uint32_t sel = B | ((B + 4) << 4);
    return __byte_perm(__byte_perm(a, b, sel), __byte_perm(c, d, sel), 0x5410);
}

// Byte permute with the full selector: a selector nibble with bit 3 set replicates the top bit of
// the selected byte over the whole result byte (the __byte_perm intrinsic keeps only 3 bits).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Byte masks (0xFF where negative) of four binary32 values / of the four bf16 values in two words.
__device__ __forceinline__ uint32_t sign_bytes_f32(float a, float b, float c, float d)
{
    const uint32_t lo = prmt(__float_as_uint(a), __float_as_uint(b), 0x00FBu);   // sign of bytes 3 and 7
    const uint32_t hi = prmt(__float_as_uint(c), __float_as_uint(d), 0x00FBu);
    return __byte_perm(lo, hi, 0x5410);
}
__device__ __forceinline__ uint32_t sign_bytes_bf16(uint32_t w01, uint32_t w23)
{
    return prmt(w01, w23, 0xFDB9u);                                              // sign of bytes 1, 3, 5, 7
}

// Four levels 0..127 in the bytes of `mag`; bytes selected by `neg` (0xFF / 0x00) are negated
// in two's complement.  0x80 - L never borrows from the next byte (L <= 127), and flipping the
// top bit turns it into 0x100 - L for L > 0 and into 0 for L = 0.
__device__ __forceinline__ uint32_t negate_bytes(uint32_t mag, uint32_t neg)
{
    const uint32_t minus = (0x80808080u - mag) ^ 0x80808080u;
    return (mag & ~neg) | (minus & neg);
}

// The same for four bytes that hold -L (0, or 0x81 .. 0xFF): where `neg` is 0xFF the byte stays,
// elsewhere it becomes L.  b ^ 0x80 = 128 - L lies in 1 .. 128, so 0x80 - (b ^ 0x80) = L borrows
// nothing from the next byte.
__device__ __forceinline__ uint32_t negated_bytes_to_signed(uint32_t minus, uint32_t neg)
{
    const uint32_t mag = 0x80808080u - (minus ^ 0x80808080u);
    return (minus & neg) | (mag & ~neg);
}

// The low nibbles of the eight bytes of (lo, hi), packed into 32 bits (byte k -> nibble k): the
// even bytes and the odd bytes are gathered into a word each, and the odd ones move up a nibble.
__device__ __forceinline__ uint32_t bytes_to_nibbles(uint32_t lo, uint32_t hi)
{
    const uint32_t even = __byte_perm(lo, hi, 0x6420), odd = __byte_perm(lo, hi, 0x7531);
    return (even & 0x0F0F0F0Fu) | ((odd << 4) & 0xF0F0F0F0u);
}

// ---------------------------------------------------------------------------------------------
// Level wire formats: bytes of one worker's level row, and where the levels of the unit of 8
// coordinates that starts at coordinate i (a multiple of 8) sit in it.  UQ_FMT_I6P keeps two
// planes per row: the low four bits of every level as nibbles (as UQ_FMT_I4X2) in the first
// stride/2 bytes, bits 4 and 5 as 2-bit fields (as UQ_FMT_I2X4) in the stride/4 bytes that follow.
// ---------------------------------------------------------------------------------------------
template <int FMT> struct LevelFmt {
    static constexpr int UB = 8 >> FMT;                                        // bytes per unit
    static __host__ __device__ __forceinline__ size_t row_bytes(int64_t stride) { return (size_t)(stride >> FMT); }
    static __host__ __device__ __forceinline__ size_t off(int64_t i) { return (size_t)(i >> FMT); }
    static __host__ __device__ __forceinline__ size_t off2(int64_t, int64_t) { return 0; }
};
template <> struct LevelFmt<UQ_FMT_I6P> {
    static constexpr int UB = 4, UB2 = 2;                                      // nibble plane, 2-bit plane
    static __host__ __device__ __forceinline__ size_t row_bytes(int64_t stride) { return ((size_t)(stride >> 1) + (size_t)(stride >> 2) + 15) & ~(size_t)15; }
    static __host__ __device__ __forceinline__ size_t off(int64_t i) { return (size_t)(i >> 1); }
    static __host__ __device__ __forceinline__ size_t off2(int64_t i, int64_t stride) { return (size_t)(stride >> 1) + (size_t)(i >> 2); }
};

// ---------------------------------------------------------------------------------------------
// the segment of a tile, found by one warp without shared memory
// ---------------------------------------------------------------------------------------------

// Smallest j in [0, nseg-1] with seg_off[j+1] > i, searched by all 32 lanes of the calling warp
// together: every step probes 32 evenly spaced entries and a ballot narrows the range 32-fold,
// so nseg <= 1024 costs two dependent loads.  The result is clamped to the table whatever the
// table holds.  Must be called by a full warp with the same arguments in every lane.
__device__ __forceinline__ int warp_find_segment(const int64_t *__restrict__ seg_off, int nseg, int64_t i)
{
    if (seg_off == nullptr) return 0;
    const int lane = threadIdx.x & 31;
    int lo = 0, hi = nseg - 1;
    while (lo < hi) {
        const int len = hi - lo + 1;
        const int step = (len + 31) >> 5;
        const int j = min(lo + (lane + 1) * step - 1, hi);           // last candidate of my slice
        const bool beyond = j >= hi || __ldg(seg_off + j + 1) > i;     // answer is at or before j
        const unsigned vote = __ballot_sync(0xFFFFFFFFu, beyond);
        const int first = __ffs(vote) - 1;                             // vote != 0: the last lane sees j >= hi
        const int nlo = lo + first * step;
        hi = min(nlo + step - 1, hi);
        lo = min(nlo, hi);
    }
    return lo;
}

// Reconstruction factor W / ((float)s * (float)M): product, then one IEEE division (W = 0 gives 0).
__device__ __forceinline__ float decode_factor(float W, int32_t s, int M)
{
    return __fdiv_rn(W, __fmul_rn((float)s, (float)M));
}

// ---------------------------------------------------------------------------------------------
// scale selection: the test |v| * inv <= s_hat as an integer compare
// ---------------------------------------------------------------------------------------------

// Largest non-negative binary32 bit pattern t with fl(t * inv) <= s_hat, or -1 if not even 0
// passes.  fl(t * inv) is non-decreasing in t, so "passes" is a prefix of the magnitudes and the
// test |v| * inv <= s_hat is the integer compare bits(|v|) <= t.  The quotient s_hat / inv lands
// within a few units of the answer; the two bounded loops settle it exactly.
__device__ __forceinline__ int32_t pass_threshold(float inv, float s_hat)
{
    if (!(inv > 0.0f)) return inv == 0.0f ? 0x7F7FFFFF : -1;       // W = 0: every finite value passes
    if (!(__fmul_rn(0.0f, inv) <= s_hat)) return -1;                // inv = Inf: 0 * Inf is NaN
    int32_t b = __float_as_int(fminf(__fdiv_rn(s_hat, inv), 3.402823466e38f));
    for (int it = 0; it < 64 && b < 0x7F7FFFFF && __fmul_rn(__int_as_float(b + 1), inv) <= s_hat; ++it) ++b;
    for (int it = 0; it < 64 && b >= 0 && !(__fmul_rn(__int_as_float(b), inv) <= s_hat); ++it) --b;
    return b;
}

}  // namespace uq
