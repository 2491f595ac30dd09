// Integer aggregation of the workers' levels and reconstruction of the average gradient:
// S_i = sum_m zeta^m_i (Algorithm 1 / 2, line "AllReduce gradients") and
// g_hat_i = W_j * S_i / (s_i * M)  (Eq. R_s after Algorithm 1, Eq. R_{s_} after Algorithm 2).
//
// The fused kernel reads the M level streams once, keeps the sums in registers and writes only
// the fp32 average (and, on request, the int32 sums).  A thread owns 16 coordinates of int8 levels
// (16 B of every worker's stream) or 32 coordinates of the packed formats (16 B of 4-bit, 8 B of
// 2-bit, 16 + 8 B of the two planes of 6-bit levels).
#include <type_traits>

#include "uq_device.cuh"

namespace uq {

struct DecodeParams {
    const void *lev;          // level rows, or int32 sums for the sums-only kernel
    const float *W;
    const int64_t *seg_off;
    const uint8_t *idx;
    float *out;               // may be NULL (aggregate only)
    int32_t *S;               // may be NULL
    int64_t d, stride;
    int32_t nseg, M;
    ScaleSet scales;          // single-scale: N = 1
    // fused parameter update (theta == NULL: none)
    float *theta;             // parameters, updated in place
    float *mom;               // momentum buffer, updated in place; NULL for plain SGD
    float lr, mu, wd;         // step size, momentum factor, weight decay
    // ROWS variant: where each worker's level row starts (rows need not be one buffer, nor all on
    // this GPU: a peer's row is read with ordinary coherent loads over NVLink); lev is unused then
    const void *rows[UQ_MAX_WORKERS];
};

// One coordinate of the update theta <- theta - lr * u with
//   u = g_hat + wd * theta (weight decay, skipped when wd == 0) and, with a momentum buffer,
//   buf <- mu * buf + u,  u = buf.   One IEEE operation per step, nothing fused.
__device__ __forceinline__ void sgd_coordinate(float g_hat, float &theta, float &buf, bool has_mom, float lr, float mu,
                                               float wd)
{
    float u = g_hat;
    if (wd != 0.0f) u = __fadd_rn(u, __fmul_rn(wd, theta));
    if (has_mom) { buf = __fadd_rn(__fmul_rn(mu, buf), u); u = buf; }
    theta = __fsub_rn(theta, __fmul_rn(lr, u));
}

template <int IDXB> __device__ __forceinline__ int index_at(const uint8_t *idx, int64_t i)
{
    if (IDXB == 8) return idx[i];
    const int per = 8 / IDXB;
    return (idx[i / per] >> ((int)(i % per) * IDXB)) & ((1 << IDXB) - 1);
}

// Sums of C coordinates held by one thread.
template <int FMT> struct Unit;

template <> struct Unit<UQ_FMT_I8> {
    static constexpr int C = 16;
    using Q = uint4;                                             // one worker's levels of the unit
    // row = start of the worker's level row, i = first coordinate of the unit; PEER: the row may be
    // another GPU's memory (coherent loads instead of the read-only path)
    template <bool PEER> static __device__ __forceinline__ Q load(const char *row, int64_t i, int64_t)
    {
        return PEER ? ld_coherent(row + i) : ld_stream(row + i);
    }
    // Bytes are biased to unsigned (x ^ 0x80) and added in 16-bit lanes: two lanes per word,
    // M <= 64 workers * 255 < 2^16.  lane layout of word w: even = bytes 0,2; odd = bytes 1,3.
    uint32_t even[4] = {0, 0, 0, 0}, odd[4] = {0, 0, 0, 0};
    __device__ __forceinline__ void add(const uint4 &q)
    {
        const uint32_t w[4] = { q.x, q.y, q.z, q.w };
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t b = w[k] ^ 0x80808080u;
            even[k] += b & 0x00FF00FFu;
            odd[k] += (b >> 8) & 0x00FF00FFu;
        }
    }
    __device__ __forceinline__ void prepare() {}
    // the sums of coordinates E0 .. E0 + 7 of the unit (E0 a multiple of 8)
    template <int E0> __device__ __forceinline__ void sums8(int M, int (&s)[8]) const
    {
        const int bias = 128 * M;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            s[4 * k + 0] = (int)(even[E0 / 4 + k] & 0xFFFFu) - bias;
            s[4 * k + 1] = (int)(odd[E0 / 4 + k] & 0xFFFFu) - bias;
            s[4 * k + 2] = (int)(even[E0 / 4 + k] >> 16) - bias;
            s[4 * k + 3] = (int)(odd[E0 / 4 + k] >> 16) - bias;
        }
    }
};

template <> struct Unit<UQ_FMT_I4X2> {
    static constexpr int C = 32;
    using Q = uint4;
    template <bool PEER> static __device__ __forceinline__ Q load(const char *row, int64_t i, int64_t)
    {
        return PEER ? ld_coherent(row + (i >> 1)) : ld_stream(row + (i >> 1));
    }
    // Nibbles are biased to unsigned (x ^ 8) and added in byte lanes for up to 16 workers
    // (16 * 15 < 256), then widened into 16-bit lanes.
    uint32_t lo8[4] = {0, 0, 0, 0}, hi8[4] = {0, 0, 0, 0};       // byte lanes: even / odd nibbles
    uint32_t acc[4][4] = {};                                    // 16-bit lanes, see finish()
    int pending = 0;
    __device__ __forceinline__ void flush()
    {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc[k][0] += lo8[k] & 0x00FF00FFu;          // nibbles 0, 4
            acc[k][1] += (lo8[k] >> 8) & 0x00FF00FFu;   // nibbles 2, 6
            acc[k][2] += hi8[k] & 0x00FF00FFu;          // nibbles 1, 5
            acc[k][3] += (hi8[k] >> 8) & 0x00FF00FFu;   // nibbles 3, 7
            lo8[k] = 0; hi8[k] = 0;
        }
        pending = 0;
    }
    __device__ __forceinline__ void add(const uint4 &q)
    {
        const uint32_t w[4] = { q.x, q.y, q.z, q.w };
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t b = w[k] ^ 0x88888888u;
            lo8[k] += b & 0x0F0F0F0Fu;
            hi8[k] += (b >> 4) & 0x0F0F0F0Fu;
        }
        if (++pending == 16) flush();
    }
    __device__ __forceinline__ void prepare() { flush(); }
    template <int E0> __device__ __forceinline__ void sums8(int M, int (&s)[8]) const
    {
        const int bias = 8 * M;
        constexpr int k = E0 / 8;
        s[0] = (int)(acc[k][0] & 0xFFFFu) - bias;
        s[4] = (int)(acc[k][0] >> 16) - bias;
        s[2] = (int)(acc[k][1] & 0xFFFFu) - bias;
        s[6] = (int)(acc[k][1] >> 16) - bias;
        s[1] = (int)(acc[k][2] & 0xFFFFu) - bias;
        s[5] = (int)(acc[k][2] >> 16) - bias;
        s[3] = (int)(acc[k][3] & 0xFFFFu) - bias;
        s[7] = (int)(acc[k][3] >> 16) - bias;
    }
};

template <> struct Unit<UQ_FMT_I2X4> {
    static constexpr int C = 32;
    using Q = uint2;
    template <bool PEER> static __device__ __forceinline__ Q load(const char *row, int64_t i, int64_t)
    {
        return PEER ? ld_coherent64(row + (i >> 2)) : ld_stream64(row + (i >> 2));
    }
    // 2-bit fields are biased to unsigned (x ^ 2, so 1..3).  The even and the odd fields of a word
    // are first added in 4-bit lanes (two masks, one shift and two additions per word and worker)
    // for up to 4 workers (4 * 3 < 16), then widened into byte lanes: field t of every byte of
    // word w goes to acc[w][t]; 64 workers * 3 < 256, so a byte lane never carries.
    uint32_t acc[2][4] = {};
    uint32_t ev4[2] = {0, 0}, od4[2] = {0, 0};                 // 4-bit lanes: fields 0, 2, .. / 1, 3, .. of each word
    int pending = 0;
    __device__ __forceinline__ void flush()
    {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            acc[k][0] += ev4[k] & 0x0F0F0F0Fu;                   // nibble 2y of the even lanes = field 4y
            acc[k][2] += (ev4[k] >> 4) & 0x0F0F0F0Fu;            // nibble 2y + 1 = field 4y + 2
            acc[k][1] += od4[k] & 0x0F0F0F0Fu;                   // field 4y + 1
            acc[k][3] += (od4[k] >> 4) & 0x0F0F0F0Fu;            // field 4y + 3
            ev4[k] = 0; od4[k] = 0;
        }
        pending = 0;
    }
    __device__ __forceinline__ void add(const uint2 &q)
    {
        const uint32_t w[2] = { q.x, q.y };
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t b = w[k] ^ 0xAAAAAAAAu;
            ev4[k] += b & 0x33333333u;
            od4[k] += (b >> 2) & 0x33333333u;
        }
        if (++pending == 4) flush();
    }
    __device__ __forceinline__ void prepare() { flush(); }
    template <int E0> __device__ __forceinline__ void sums8(int M, int (&s)[8]) const
    {
        const int bias = 2 * M;
        constexpr int k = E0 / 16, y0 = (E0 % 16) / 4;
#pragma unroll
        for (int y = 0; y < 2; ++y)
#pragma unroll
            for (int t = 0; t < 4; ++t) s[4 * y + t] = (int)((acc[k][t] >> (8 * (y0 + y))) & 0xFFu) - bias;
    }
};

// 6-bit levels in two planes: zeta = 16 * sx2(bits 4..5) + (bits 0..3), so the sum over workers is
// 16 * (sum of the 2-bit plane read as signed) + (sum of the nibble plane read as unsigned).
template <> struct Unit<UQ_FMT_I6P> {
    static constexpr int C = 32;
    struct Q { uint4 n; uint2 c; };
    template <bool PEER> static __device__ __forceinline__ Q load(const char *row, int64_t i, int64_t stride)
    {
        Q q;
        q.n = PEER ? ld_coherent(row + (i >> 1)) : ld_stream(row + (i >> 1));
        q.c = PEER ? ld_coherent64(row + (stride >> 1) + (i >> 2)) : ld_stream64(row + (stride >> 1) + (i >> 2));
        return q;
    }
    uint32_t lo8[4] = {0, 0, 0, 0}, hi8[4] = {0, 0, 0, 0};       // nibble plane, byte lanes: even / odd nibbles
    uint32_t acc[4][4] = {};                                    // nibble plane, 16-bit lanes
    uint32_t cr[2][4] = {};                                     // 2-bit plane, byte lanes (biased by 2)
    int pending = 0;
    __device__ __forceinline__ void flush()
    {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc[k][0] += lo8[k] & 0x00FF00FFu;
            acc[k][1] += (lo8[k] >> 8) & 0x00FF00FFu;
            acc[k][2] += hi8[k] & 0x00FF00FFu;
            acc[k][3] += (hi8[k] >> 8) & 0x00FF00FFu;
            lo8[k] = 0; hi8[k] = 0;
        }
        pending = 0;
    }
    __device__ __forceinline__ void add(const Q &q)
    {
        const uint32_t w[4] = { q.n.x, q.n.y, q.n.z, q.n.w };
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            lo8[k] += w[k] & 0x0F0F0F0Fu;                        // unsigned nibbles: 16 * 15 < 256
            hi8[k] += (w[k] >> 4) & 0x0F0F0F0Fu;
        }
        if (++pending == 16) flush();
        const uint32_t c[2] = { q.c.x, q.c.y };
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t b = c[k] ^ 0xAAAAAAAAu;
#pragma unroll
            for (int t = 0; t < 4; ++t) cr[k][t] += (b >> (2 * t)) & 0x03030303u;
        }
    }
    __device__ __forceinline__ void prepare() { flush(); }
    template <int E0> __device__ __forceinline__ void sums8(int M, int (&s)[8]) const
    {
        constexpr int kn = E0 / 8;                                   // word of the nibble plane
        int lo[8];
        lo[0] = (int)(acc[kn][0] & 0xFFFFu); lo[4] = (int)(acc[kn][0] >> 16);
        lo[2] = (int)(acc[kn][1] & 0xFFFFu); lo[6] = (int)(acc[kn][1] >> 16);
        lo[1] = (int)(acc[kn][2] & 0xFFFFu); lo[5] = (int)(acc[kn][2] >> 16);
        lo[3] = (int)(acc[kn][3] & 0xFFFFu); lo[7] = (int)(acc[kn][3] >> 16);
        const int bias = 2 * M;
        constexpr int k = E0 / 16, y0 = (E0 % 16) / 4;                // word and bytes of the 2-bit plane
#pragma unroll
        for (int y = 0; y < 2; ++y)
#pragma unroll
            for (int t = 0; t < 4; ++t)
                s[4 * y + t] = 16 * ((int)((cr[k][t] >> (8 * (y0 + y))) & 0xFFu) - bias) + lo[4 * y + t];
    }
};

// UPDATE selects the variant that also applies the parameter update (kept apart so that the plain
// reconstruction keeps its register count).
template <int FMT, int IDXB, bool UPDATE, bool ROWS = false>
__global__ void __launch_bounds__(kThreads) aggregate_decode_kernel(const __grid_constant__ DecodeParams p)
{
    grid_dependency_prologue();
    using U = Unit<FMT>;
    constexpr int C = U::C;
    constexpr bool MULTI = IDXB != 0;
    constexpr int IB = MULTI ? IDXB : 8;
    constexpr int WORDS = C * IB >= 32 ? C * IB / 32 : 1;           // idx words per thread (a half word for 16 bits)
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t i = ((int64_t)blockIdx.x * kThreads + tid) * C;  // my first coordinate
    const int64_t row0 = i - (int64_t)lane * C;                    // my warp's first coordinate
    if (row0 >= p.d) return;                                       // warp-uniform
    const bool active = i < p.d;
    using Q = typename U::Q;
    const size_t row_bytes = LevelFmt<FMT>::row_bytes(p.stride);

    U unit;
    uint32_t kw[WORDS];
    if (active) {
        int m = 0;
        for (; m + 8 <= p.M; m += 8) {          // eight workers' loads in flight
            Q q[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                q[k] = U::template load<ROWS>(ROWS ? (const char *)p.rows[m + k] : (const char *)p.lev + (size_t)(m + k) * row_bytes,
                                              i, p.stride);
#pragma unroll
            for (int k = 0; k < 8; ++k) unit.add(q[k]);
        }
        for (; m < p.M; ++m)
            unit.add(U::template load<ROWS>(ROWS ? (const char *)p.rows[m] : (const char *)p.lev + (size_t)m * row_bytes, i, p.stride));
        if (MULTI && p.out != nullptr) {
            // idx bits of coordinates i..i+C-1 start at byte i*IB/8 (a multiple of 4 bytes, of 2 for 16 bits)
            if (C * IB == 16) {
                kw[0] = __ldg((const uint16_t *)(p.idx + (size_t)i * IB / 8));
            } else {
                const uint32_t *ip = (const uint32_t *)(p.idx + (size_t)i * IB / 8);
#pragma unroll
                for (int w = 0; w < WORDS; ++w) kw[w] = __ldg(ip + w);
            }
        }
    }

    // The sums leave the accumulators eight coordinates at a time: each group is reconstructed,
    // stored (256 bits per array) and forgotten, which keeps the registers of a thread low enough for
    // more CTAs per SM than 32 sums and 32 values held at once would allow.
    unit.prepare();
    const bool full = i + C <= p.d;
    const bool want_values = p.out != nullptr || UPDATE;
    // every warp looks up the segment of its own row of 32*C coordinates; lane k holds the
    // reconstruction factor of scale k (single-scale: every lane holds the same factor)
    const int64_t row1 = min(row0 + 32 * C, p.d);
    int j = 0;
    bool uniform = true;
    float c_lane = 0.0f;
    if (want_values) {
        j = warp_find_segment(p.seg_off, p.nseg, row0);
        uniform = segment_end(p.seg_off, p.nseg, j, p.d) >= row1;
        if (uniform) c_lane = decode_factor(__ldg(p.W + j), p.scales.s[lane & (UQ_MAX_SCALES - 1)], p.M);
    }
    const bool has_mom = UPDATE && p.mom != nullptr;
    auto group = [&](auto e0_tag) {
        constexpr int E0 = decltype(e0_tag)::value;
        int s[8];
        unit.template sums8<E0>(p.M, s);
        if (p.S != nullptr && active) {
            if (full) {
                st_stream256(p.S + i + E0, *(const uint32_t(*)[8])s);
            } else {
                for (int e = 0; e < 8; ++e)
                    if (i + E0 + e < p.d) p.S[i + E0 + e] = s[e];
            }
        }
        if (!want_values) return;
        float r[8];
        if (uniform) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int k = MULTI ? (kw[((E0 + e) * IB) >> 5] >> (((E0 + e) * IB) & 31)) & ((1 << IB) - 1) : 0;
                const float c = MULTI ? __shfl_sync(0xFFFFFFFFu, c_lane, active ? k : 0) : c_lane;
                r[e] = __fmul_rn((float)s[e], c);
            }
        } else if (active) {                       // a boundary inside the row: walk on from segment j
            for (int e = 0; e < 8; ++e) {
                r[e] = 0.0f;
                if (i + E0 + e >= p.d) continue;
                j = advance_segment(p.seg_off, p.nseg, j, i + E0 + e);
                const int k = MULTI ? index_at<IB>(p.idx, i + E0 + e) : 0;
                r[e] = __fmul_rn((float)s[e], decode_factor(__ldg(p.W + j), p.scales.s[k & (UQ_MAX_SCALES - 1)], p.M));
            }
        }
        if (!active) return;
        if (UPDATE) {
            // Algorithm 1 / 2, line "Update parameters", fused: the reconstructed gradient goes straight
            // from registers into the parameters (and the momentum buffer), 8 coordinates as one
            // 256-bit access per array: a lane's 32 bytes are one whole sector
            if (full) {
                float th[8], bf[8] = {};
                ld256(p.theta + i + E0, th);
                if (has_mom) ld256(p.mom + i + E0, bf);
#pragma unroll
                for (int t = 0; t < 8; ++t) sgd_coordinate(r[t], th[t], bf[t], has_mom, p.lr, p.mu, p.wd);
                st256(p.theta + i + E0, th);
                if (has_mom) st256(p.mom + i + E0, bf);
            } else {
                for (int e = 0; e < 8; ++e) {
                    if (i + E0 + e >= p.d) break;
                    float th = p.theta[i + E0 + e], bf = has_mom ? p.mom[i + E0 + e] : 0.0f;
                    sgd_coordinate(r[e], th, bf, has_mom, p.lr, p.mu, p.wd);
                    p.theta[i + E0 + e] = th;
                    if (has_mom) p.mom[i + E0 + e] = bf;
                }
            }
        }
        if (p.out == nullptr) return;
        if (full) {
            st_stream256(p.out + i + E0, *(const uint32_t(*)[8])r);
        } else {
            for (int e = 0; e < 8; ++e)
                if (i + E0 + e < p.d) p.out[i + E0 + e] = r[e];
        }
    };
    group(std::integral_constant<int, 0>());
    group(std::integral_constant<int, 8>());
    if (C > 16) {
        group(std::integral_constant<int, (C > 16 ? 16 : 0)>());
        group(std::integral_constant<int, (C > 16 ? 24 : 0)>());
    }
}

// Reconstruction from already-summed levels (one thread per 4 coordinates).
template <int IDXB>
__global__ void __launch_bounds__(kThreads) decode_sums_kernel(const DecodeParams p)
{
    grid_dependency_prologue();
    constexpr bool MULTI = IDXB != 0;
    const int64_t i = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 4;
    if (i >= p.d) return;
    const int32_t *S = (const int32_t *)p.lev;
    int s[4] = {0, 0, 0, 0};
    const bool full = i + 4 <= p.d;
    if (full) {
        const int4 q = *(const int4 *)(S + i);
        s[0] = q.x; s[1] = q.y; s[2] = q.z; s[3] = q.w;
    } else {
        for (int e = 0; e < 4; ++e)
            if (i + e < p.d) s[e] = S[i + e];
    }
    float r[4];
    int j = find_segment(p.seg_off, p.nseg, i);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        r[e] = 0.0f;
        if (i + e >= p.d) continue;
        j = advance_segment(p.seg_off, p.nseg, j, i + e);
        const int k = MULTI ? index_at<MULTI ? IDXB : 8>(p.idx, i + e) : 0;
        r[e] = __fmul_rn((float)s[e], decode_factor(__ldg(p.W + j), p.scales.s[k & (UQ_MAX_SCALES - 1)], p.M));
    }
    if (full) *(float4 *)(p.out + i) = make_float4(r[0], r[1], r[2], r[3]);
    else
        for (int e = 0; e < 4; ++e)
            if (i + e < p.d) p.out[i + e] = r[e];
}

template <int FMT>
static cudaError_t dispatch_levels(const DecodeParams &p, int idx_bits, cudaStream_t st, bool rows = false)
{
    constexpr int TILE = kThreads * Unit<FMT>::C;
    const int64_t blocks = (p.d + TILE - 1) / TILE;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const unsigned nb = (unsigned)blocks;
    if (rows) {
        switch (idx_bits) {
        case 0: launch_k(aggregate_decode_kernel<FMT, 0, false, true>, nb, kThreads, st, p); break;
        case 1: launch_k(aggregate_decode_kernel<FMT, 1, false, true>, nb, kThreads, st, p); break;
        case 2: launch_k(aggregate_decode_kernel<FMT, 2, false, true>, nb, kThreads, st, p); break;
        case 4: launch_k(aggregate_decode_kernel<FMT, 4, false, true>, nb, kThreads, st, p); break;
        default: launch_k(aggregate_decode_kernel<FMT, 8, false, true>, nb, kThreads, st, p); break;
        }
        return cudaGetLastError();
    }
    if (p.theta != nullptr) {
        switch (idx_bits) {
        case 0: launch_k(aggregate_decode_kernel<FMT, 0, true>, nb, kThreads, st, p); break;
        case 1: launch_k(aggregate_decode_kernel<FMT, 1, true>, nb, kThreads, st, p); break;
        case 2: launch_k(aggregate_decode_kernel<FMT, 2, true>, nb, kThreads, st, p); break;
        case 4: launch_k(aggregate_decode_kernel<FMT, 4, true>, nb, kThreads, st, p); break;
        default: launch_k(aggregate_decode_kernel<FMT, 8, true>, nb, kThreads, st, p); break;
        }
        return cudaGetLastError();
    }
    switch (idx_bits) {
    case 0: launch_k(aggregate_decode_kernel<FMT, 0, false>, nb, kThreads, st, p); break;
    case 1: launch_k(aggregate_decode_kernel<FMT, 1, false>, nb, kThreads, st, p); break;
    case 2: launch_k(aggregate_decode_kernel<FMT, 2, false>, nb, kThreads, st, p); break;
    case 4: launch_k(aggregate_decode_kernel<FMT, 4, false>, nb, kThreads, st, p); break;
    default: launch_k(aggregate_decode_kernel<FMT, 8, false>, nb, kThreads, st, p); break;
    }
    return cudaGetLastError();
}

// out == NULL: aggregate only.  idx_bits == 0: single scale (scales = {s}).
cudaError_t launch_aggregate_decode(const uq_layout &L, const void *lev, int fmt, const float *W,
                                    const ScaleSet &scales, const uint8_t *idx, int idx_bits, float *out,
                                    int32_t *S, cudaStream_t st, float *theta, float *mom, float lr, float mu,
                                    float wd)
{
    DecodeParams p = DecodeParams();
    p.lev = lev; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.out = out; p.S = S;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M; p.scales = scales;
    p.theta = theta; p.mom = mom; p.lr = lr; p.mu = mu; p.wd = wd;
    if (fmt == UQ_FMT_I8) return dispatch_levels<UQ_FMT_I8>(p, idx_bits, st);
    if (fmt == UQ_FMT_I4X2) return dispatch_levels<UQ_FMT_I4X2>(p, idx_bits, st);
    if (fmt == UQ_FMT_I2X4) return dispatch_levels<UQ_FMT_I2X4>(p, idx_bits, st);
    return dispatch_levels<UQ_FMT_I6P>(p, idx_bits, st);
}

// The same with the level rows given one by one (lev_rows[m] = start of worker m's row).
cudaError_t launch_aggregate_decode_rows(const uq_layout &L, const void *const *lev_rows, int fmt, const float *W,
                                         const ScaleSet &scales, const uint8_t *idx, int idx_bits, float *out,
                                         int32_t *S, cudaStream_t st)
{
    DecodeParams p = DecodeParams();
    p.lev = nullptr; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.out = out; p.S = S;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M; p.scales = scales;
    p.theta = nullptr; p.mom = nullptr; p.lr = p.mu = p.wd = 0.0f;
    for (int m = 0; m < UQ_MAX_WORKERS; ++m) p.rows[m] = m < L.M ? lev_rows[m] : nullptr;
    if (fmt == UQ_FMT_I8) return dispatch_levels<UQ_FMT_I8>(p, idx_bits, st, true);
    if (fmt == UQ_FMT_I4X2) return dispatch_levels<UQ_FMT_I4X2>(p, idx_bits, st, true);
    if (fmt == UQ_FMT_I2X4) return dispatch_levels<UQ_FMT_I2X4>(p, idx_bits, st, true);
    return dispatch_levels<UQ_FMT_I6P>(p, idx_bits, st, true);
}

cudaError_t launch_decode_sums(const uq_layout &L, const int32_t *S, const float *W, const ScaleSet &scales,
                               const uint8_t *idx, int idx_bits, float *out, cudaStream_t st)
{
    DecodeParams p = DecodeParams();
    p.lev = S; p.W = W; p.seg_off = L.seg_off; p.idx = idx; p.out = out; p.S = nullptr;
    p.theta = nullptr; p.mom = nullptr; p.lr = p.mu = p.wd = 0.0f;
    p.d = L.d; p.stride = L.worker_stride; p.nseg = L.nseg; p.M = L.M; p.scales = scales;
    const int64_t blocks = (L.d + kThreads * 4 - 1) / (kThreads * 4);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const unsigned nb = (unsigned)blocks;
    switch (idx_bits) {
    case 0: launch_k(decode_sums_kernel<0>, nb, kThreads, st, p); break;
    case 1: launch_k(decode_sums_kernel<1>, nb, kThreads, st, p); break;
    case 2: launch_k(decode_sums_kernel<2>, nb, kThreads, st, p); break;
    case 4: launch_k(decode_sums_kernel<4>, nb, kThreads, st, p); break;
    default: launch_k(decode_sums_kernel<8>, nb, kThreads, st, p); break;
    }
    return cudaGetLastError();
}

}  // namespace uq
