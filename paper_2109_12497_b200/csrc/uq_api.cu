// The C ABI declared in include/uq.h: argument validation on the host, then kernel launches.
// No allocation, no synchronization, no state besides a thread-local last CUDA error.
#include "uq_device.cuh"

namespace uq {
int64_t norm_tiles(int64_t d);
cudaError_t launch_agree_scale(const uq_layout &L, const void *g, int norm, float *W, uint32_t *status,
                               void *workspace, cudaStream_t st);
cudaError_t launch_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                          uint32_t *status, cudaStream_t st);
cudaError_t launch_select(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                          int idx_bits, uint8_t *idx, uint32_t *status, cudaStream_t st);
cudaError_t launch_aggregate_decode(const uq_layout &L, const void *lev, int fmt, const float *W,
                                    const ScaleSet &scales, const uint8_t *idx, int idx_bits, float *out,
                                    int32_t *S, cudaStream_t st, float *theta = nullptr, float *mom = nullptr,
                                    float lr = 0.0f, float mu = 0.0f, float wd = 0.0f);
cudaError_t launch_aggregate_decode_rows(const uq_layout &L, const void *const *lev_rows, int fmt, const float *W,
                                         const ScaleSet &scales, const uint8_t *idx, int idx_bits, float *out,
                                         int32_t *S, cudaStream_t st);
cudaError_t launch_decode_sums(const uq_layout &L, const int32_t *S, const float *W, const ScaleSet &scales,
                               const uint8_t *idx, int idx_bits, float *out, cudaStream_t st);
cudaError_t launch_select_encode_decode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                                        int idx_bits, uint64_t seed, uint8_t *idx, void *lev, float *out, uint32_t *status,
                                        cudaStream_t st);
bool encode_decode_fused(const uq_layout &L, int fmt, int rng_bits);
cudaError_t launch_encode_decode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales,
                                 const uint8_t *idx, int idx_bits, uint64_t seed, void *lev, float *out, uint32_t *status,
                                 cudaStream_t st);
cudaError_t launch_select_encode(const uq_layout &L, const void *g, const float *W, const ScaleSet &scales, int idx_bits,
                                 uint64_t seed, int rng_bits, int fmt, uint8_t *idx, void *lev, uint32_t *status,
                                 cudaStream_t st);
cudaError_t launch_index_min(const uint8_t *rows, int R, int64_t row_bytes, int64_t nbytes, int idx_bits, uint8_t *idx,
                             cudaStream_t st);
cudaError_t launch_randk_gather(const uq_layout &L, const void *g, int64_t K, uint64_t seed, int64_t *sel,
                                void *gk, int64_t gk_stride, uint32_t *status, cudaStream_t st);
cudaError_t launch_randk_scatter(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *dst, bool update,
                                 float lr, uint32_t *status, cudaStream_t st);
bool small_step_supported(const uq_layout &L, int fmt);
size_t small_workspace_bytes();
cudaError_t launch_small_step(const uq_layout &L, const void *g, int norm, int s, uint64_t seed, int rng_bits, int fmt,
                              float *W, void *lev, float *out, int32_t *S, uint32_t *status, void *workspace,
                              cudaStream_t st);
cudaError_t launch_small_step_multi(const uq_layout &L, const void *g, int norm, const ScaleSet &scales, int idx_bits,
                                    uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev, float *out,
                                    int32_t *S, uint32_t *status, void *workspace, cudaStream_t st);
}  // namespace uq

namespace {
thread_local int g_last_cuda_error = 0;
}

namespace uq {
// UQ_OK, or UQ_ERR_CUDA with the code kept for uq_last_cuda_error() (every entry point of the
// library reports its CUDA failures through here, whichever file it lives in).
int record_cuda_error(cudaError_t e)
{
    if (e == cudaSuccess) return UQ_OK;
    g_last_cuda_error = (int)e;
    return UQ_ERR_CUDA;
}
}  // namespace uq

namespace {

int finish(cudaError_t e) { return uq::record_cuda_error(e); }

bool aligned(const void *p, size_t a) { return ((uintptr_t)p & (a - 1)) == 0; }

bool layout_ok(const uq_layout *L)
{
    if (L == nullptr) return false;
    if (L->d < 0 || L->M < 1 || L->M > UQ_MAX_WORKERS || L->nseg < 1 || L->worker0 < 0 || L->worker0 > 0x7FFFFFFF - L->M) return false;
    if (L->dtype != UQ_F32 && L->dtype != UQ_BF16) return false;
    if (L->worker_stride < L->d || (L->worker_stride & 31) != 0) return false;
    if (L->seg_off == nullptr && L->nseg != 1) return false;
    if (L->seg_off != nullptr && !aligned(L->seg_off, 8)) return false;
    if (L->d > (int64_t)1 << 40) return false;
    if (L->coord0 < 0 || (L->coord0 & 7) != 0 || L->coord0 > (int64_t)1 << 40) return false;
    return true;
}

bool idx_bits_ok(int b) { return b == 1 || b == 2 || b == 4 || b == 8; }

bool fmt_known(int fmt) { return fmt == UQ_FMT_I8 || fmt == UQ_FMT_I4X2 || fmt == UQ_FMT_I2X4 || fmt == UQ_FMT_I6P; }

bool fmt_ok(int fmt, int s_hat)
{
    if (fmt == UQ_FMT_I8) return s_hat >= 1 && s_hat <= 127;
    if (fmt == UQ_FMT_I4X2) return s_hat >= 1 && s_hat <= 7;
    if (fmt == UQ_FMT_I2X4) return s_hat == 1;
    if (fmt == UQ_FMT_I6P) return s_hat >= 1 && s_hat <= 31;
    return false;
}

// Copies an ascending scale set into the kernel-parameter form; false if it is not valid.
bool scales_ok(const int32_t *scales, int N, int idx_bits, uq::ScaleSet *out)
{
    if (scales == nullptr || N < 1 || N > UQ_MAX_SCALES) return false;
    if (!idx_bits_ok(idx_bits)) return false;
    if (idx_bits < 8 && N > (1 << idx_bits)) return false;
    for (int k = 0; k < N; ++k) {
        if (scales[k] < 1) return false;
        if (k > 0 && scales[k] <= scales[k - 1]) return false;
        out->s[k] = scales[k];
    }
    for (int k = N; k < UQ_MAX_SCALES; ++k) out->s[k] = scales[N - 1];
    out->N = N;
    return true;
}

uq::ScaleSet single_scale(int s)
{
    uq::ScaleSet set;
    for (int k = 0; k < UQ_MAX_SCALES; ++k) set.s[k] = s;
    set.N = 1;
    return set;
}

}  // namespace

extern "C" {

int uq_version(void) { return 100; }

int uq_last_cuda_error(void) { return g_last_cuda_error; }

const char *uq_error_string(int code)
{
    switch (code) {
    case UQ_OK: return "ok";
    case UQ_ERR_BAD_ARG: return "bad argument";
    case UQ_ERR_CUDA: return "CUDA launch failed (see uq_last_cuda_error)";
    case UQ_ERR_UNSUPPORTED: return "unsupported combination";
    case UQ_ERR_WORKSPACE: return "workspace missing or too small";
    default: return "unknown error code";
    }
}

size_t uq_workspace_bytes(const uq_layout *L)
{
    if (!layout_ok(L)) return 0;
    return (size_t)L->M * (size_t)(uq::norm_tiles(L->d) + L->nseg) * sizeof(double);
}

size_t uq_index_bytes(const uq_layout *L, int idx_bits)
{
    if (!layout_ok(L) || !idx_bits_ok(idx_bits)) return 0;
    return (size_t)L->worker_stride * (size_t)idx_bits / 8;
}

int uq_agree_scale(const uq_layout *L, const void *g, int norm, float *W, uint32_t *status, void *workspace,
                   size_t workspace_bytes, void *stream)
{
    if (!layout_ok(L) || W == nullptr || !aligned(W, 4) || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (norm != UQ_NORM_L2 && norm != UQ_NORM_LINF) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || !aligned(g, 16))) return UQ_ERR_BAD_ARG;
    if (workspace == nullptr || !aligned(workspace, 8) || workspace_bytes < uq_workspace_bytes(L))
        return UQ_ERR_WORKSPACE;
    return finish(uq::launch_agree_scale(*L, g, norm, W, status, workspace, (cudaStream_t)stream));
}

int uq_encode_single(const uq_layout *L, const void *g, const float *W, int s, uint64_t seed, int rng_bits,
                     int fmt, void *lev, uint32_t *status, void *stream)
{
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (!fmt_ok(fmt, s) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || !aligned(g, 16) || !aligned(lev, 16)))
        return UQ_ERR_BAD_ARG;
    return finish(uq::launch_encode(*L, g, W, single_scale(s), nullptr, 0, seed, rng_bits, fmt, lev, status,
                                    (cudaStream_t)stream));
}

int uq_select_scale_multi(const uq_layout *L, const void *g, const float *W, const int32_t *scales, int N,
                          int idx_bits, uint8_t *idx, uint32_t *status, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || idx == nullptr || !aligned(g, 16) || !aligned(idx, 16)))
        return UQ_ERR_BAD_ARG;
    return finish(uq::launch_select(*L, g, W, set, idx_bits, idx, status, (cudaStream_t)stream));
}

int uq_encode_multi(const uq_layout *L, const void *g, const float *W, const int32_t *scales, int N,
                    const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev,
                    uint32_t *status, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
    if (!fmt_ok(fmt, set.s[0]) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || idx == nullptr || !aligned(g, 16) || !aligned(lev, 16) ||
                     !aligned(idx, 16)))
        return UQ_ERR_BAD_ARG;
    return finish(uq::launch_encode(*L, g, W, set, idx, idx_bits, seed, rng_bits, fmt, lev, status,
                                    (cudaStream_t)stream));
}

int uq_select_encode_multi(const uq_layout *L, const void *g, const float *W, const int32_t *scales, int N,
                           int idx_bits, uint64_t seed, int rng_bits, int fmt, uint8_t *idx, void *lev,
                           uint32_t *status, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
    if (!fmt_ok(fmt, set.s[0]) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || idx == nullptr || !aligned(g, 16) || !aligned(lev, 16) ||
                     !aligned(idx, 16)))
        return UQ_ERR_BAD_ARG;
    return finish(uq::launch_select_encode(*L, g, W, set, idx_bits, seed, rng_bits, fmt, idx, lev, status,
                                           (cudaStream_t)stream));
}

int uq_aggregate(const uq_layout *L, const void *lev, int fmt, int32_t *S, void *stream)
{
    if (!layout_ok(L) || !fmt_known(fmt)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (lev == nullptr || S == nullptr || !aligned(lev, 16) || !aligned(S, 32)))
        return UQ_ERR_BAD_ARG;
    return finish(uq::launch_aggregate_decode(*L, lev, fmt, nullptr, single_scale(1), nullptr, 0, nullptr, S,
                                              (cudaStream_t)stream));
}

int uq_decode(const uq_layout *L, const void *src, int src_kind, int fmt, const float *W, int s,
              const int32_t *scales, int N, const uint8_t *idx, int idx_bits, float *out, int32_t *S_opt,
              void *stream)
{
    if (!layout_ok(L) || W == nullptr) return UQ_ERR_BAD_ARG;
    if (src_kind != UQ_SRC_LEVELS && src_kind != UQ_SRC_SUMS) return UQ_ERR_BAD_ARG;
    uq::ScaleSet set;
    if (scales != nullptr) {
        if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
        if (L->d > 0 && (idx == nullptr || !aligned(idx, 16))) return UQ_ERR_BAD_ARG;
    } else {
        if (s < 1) return UQ_ERR_BAD_ARG;
        set = single_scale(s);
        idx_bits = 0;
        idx = nullptr;
    }
    if (L->d > 0 && (src == nullptr || out == nullptr || !aligned(src, 16) || !aligned(out, 32)))
        return UQ_ERR_BAD_ARG;
    if (src_kind == UQ_SRC_SUMS)
        return finish(uq::launch_decode_sums(*L, (const int32_t *)src, W, set, idx, idx_bits, out,
                                             (cudaStream_t)stream));
    if (!fmt_known(fmt)) return UQ_ERR_BAD_ARG;
    if (S_opt != nullptr && !aligned(S_opt, 32)) return UQ_ERR_BAD_ARG;
    return finish(uq::launch_aggregate_decode(*L, src, fmt, W, set, idx, idx_bits, out, S_opt,
                                              (cudaStream_t)stream));
}

int uq_encode_decode(const uq_layout *L, const void *g, const float *W, int s, const int32_t *scales, int N,
                     const uint8_t *idx, int idx_bits, uint64_t seed, int rng_bits, int fmt, void *lev, float *out,
                     uint32_t *status, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (scales != nullptr) {
        if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
        if (L->d > 0 && (idx == nullptr || !aligned(idx, 16))) return UQ_ERR_BAD_ARG;
    } else {
        if (s < 1) return UQ_ERR_BAD_ARG;
        set = single_scale(s);
        idx_bits = 0;
        idx = nullptr;
    }
    if (!fmt_ok(fmt, set.s[0]) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || out == nullptr || !aligned(g, 16) || !aligned(lev, 16) ||
                     !aligned(out, 32)))
        return UQ_ERR_BAD_ARG;
    if (uq::encode_decode_fused(*L, fmt, rng_bits))
        return finish(uq::launch_encode_decode(*L, g, W, set, idx, idx_bits, seed, lev, out, status, (cudaStream_t)stream));
    const cudaError_t e = uq::launch_encode(*L, g, W, set, idx, idx_bits, seed, rng_bits, fmt, lev, status,
                                            (cudaStream_t)stream);
    if (e != cudaSuccess) return finish(e);
    return finish(uq::launch_aggregate_decode(*L, lev, fmt, W, set, idx, idx_bits, out, nullptr, (cudaStream_t)stream));
}

int uq_select_encode_decode_multi(const uq_layout *L, const void *g, const float *W, const int32_t *scales, int N,
                                  int idx_bits, uint64_t seed, int rng_bits, int fmt, uint8_t *idx, void *lev, float *out,
                                  uint32_t *status, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
    if (!fmt_ok(fmt, set.s[0]) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || idx == nullptr || out == nullptr || !aligned(g, 16) ||
                     !aligned(lev, 16) || !aligned(idx, 16) || !aligned(out, 32)))
        return UQ_ERR_BAD_ARG;
    if (uq::encode_decode_fused(*L, fmt, rng_bits))
        return finish(uq::launch_select_encode_decode(*L, g, W, set, idx_bits, seed, idx, lev, out, status,
                                                      (cudaStream_t)stream));
    const cudaError_t e = uq::launch_select_encode(*L, g, W, set, idx_bits, seed, rng_bits, fmt, idx, lev, status,
                                                   (cudaStream_t)stream);
    if (e != cudaSuccess) return finish(e);
    return finish(uq::launch_aggregate_decode(*L, lev, fmt, W, set, idx, idx_bits, out, nullptr, (cudaStream_t)stream));
}

int uq_decode_rows(const uq_layout *L, const void *const *lev_rows, int fmt, const float *W, int s,
                   const int32_t *scales, int N, const uint8_t *idx, int idx_bits, float *out, int32_t *S_opt,
                   void *stream)
{
    if (!layout_ok(L) || W == nullptr || lev_rows == nullptr || !fmt_known(fmt)) return UQ_ERR_BAD_ARG;
    uq::ScaleSet set;
    if (scales != nullptr) {
        if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
        if (L->d > 0 && (idx == nullptr || !aligned(idx, 16))) return UQ_ERR_BAD_ARG;
    } else {
        if (s < 1) return UQ_ERR_BAD_ARG;
        set = single_scale(s);
        idx_bits = 0;
        idx = nullptr;
    }
    if (L->d > 0) {
        if (out == nullptr || !aligned(out, 32) || !aligned(S_opt, 32)) return UQ_ERR_BAD_ARG;
        for (int m = 0; m < L->M; ++m)
            if (lev_rows[m] == nullptr || !aligned(lev_rows[m], 16)) return UQ_ERR_BAD_ARG;
    }
    return finish(uq::launch_aggregate_decode_rows(*L, lev_rows, fmt, W, set, idx, idx_bits, out, S_opt,
                                                   (cudaStream_t)stream));
}

int uq_decode_update(const uq_layout *L, const void *lev, int fmt, const float *W, int s, const int32_t *scales,
                     int N, const uint8_t *idx, int idx_bits, float *theta, float *momentum, float lr, float mu,
                     float wd, float *out_opt, void *stream)
{
    if (!layout_ok(L) || W == nullptr || !fmt_known(fmt)) return UQ_ERR_BAD_ARG;
    if (!(lr == lr) || !(mu == mu) || !(wd == wd)) return UQ_ERR_BAD_ARG;                  // NaN hyper-parameters
    uq::ScaleSet set;
    if (scales != nullptr) {
        if (!scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
        if (L->d > 0 && (idx == nullptr || !aligned(idx, 16))) return UQ_ERR_BAD_ARG;
    } else {
        if (s < 1) return UQ_ERR_BAD_ARG;
        set = single_scale(s);
        idx_bits = 0;
        idx = nullptr;
    }
    if (L->d > 0 && (lev == nullptr || theta == nullptr || !aligned(lev, 16) || !aligned(theta, 32))) return UQ_ERR_BAD_ARG;
    if (!aligned(momentum, 32) || !aligned(out_opt, 32)) return UQ_ERR_BAD_ARG;
    if (L->d == 0) return UQ_OK;
    return finish(uq::launch_aggregate_decode(*L, lev, fmt, W, set, idx, idx_bits, out_opt, nullptr, (cudaStream_t)stream,
                                              theta, momentum, lr, mu, wd));
}

int uq_step(const uq_layout *L, const void *g, int norm, int s, const int32_t *scales, int N, int idx_bits,
            uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev, float *out, int32_t *S_opt,
            uint32_t *status, void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = uq_agree_scale(L, g, norm, W, status, workspace, workspace_bytes, stream);
    if (rc != UQ_OK) return rc;
    if (scales != nullptr) {
        // nobody wants the integer sums, and the encoder can select, add up and reconstruct itself: the
        // rest of the step is one kernel
        if (S_opt == nullptr && layout_ok(L) && uq::encode_decode_fused(*L, fmt, rng_bits))
            return uq_select_encode_decode_multi(L, g, W, scales, N, idx_bits, seed, rng_bits, fmt, idx, lev, out, status,
                                                 stream);
        rc = uq_select_scale_multi(L, g, W, scales, N, idx_bits, idx, status, stream);
        if (rc != UQ_OK) return rc;
    }
    if (S_opt == nullptr)       // nobody wants the integer sums: the encoder may add up and reconstruct itself
        return uq_encode_decode(L, g, W, s, scales, N, idx, idx_bits, seed, rng_bits, fmt, lev, out, status, stream);
    if (scales != nullptr)
        rc = uq_encode_multi(L, g, W, scales, N, idx, idx_bits, seed, rng_bits, fmt, lev, status, stream);
    else
        rc = uq_encode_single(L, g, W, s, seed, rng_bits, fmt, lev, status, stream);
    if (rc != UQ_OK) return rc;
    return uq_decode(L, lev, UQ_SRC_LEVELS, fmt, W, s, scales, N, idx, idx_bits, out, S_opt, stream);
}

size_t uq_workspace_bytes_small(void) { return uq::small_workspace_bytes(); }

int uq_step_small(const uq_layout *L, const void *g, int norm, int s, const int32_t *scales, int N, int idx_bits,
                  uint64_t seed, int rng_bits, int fmt, float *W, uint8_t *idx, void *lev, float *out, int32_t *S_opt,
                  uint32_t *status, void *workspace, size_t workspace_bytes, void *stream)
{
    uq::ScaleSet set;
    if (!layout_ok(L) || W == nullptr || !aligned(W, 4) || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (status == nullptr) return UQ_ERR_BAD_ARG;      // a wait that runs out must be able to say so
    if (norm != UQ_NORM_L2 && norm != UQ_NORM_LINF) return UQ_ERR_BAD_ARG;
    if (scales != nullptr && !scales_ok(scales, N, idx_bits, &set)) return UQ_ERR_BAD_ARG;
    if (!fmt_ok(fmt, scales != nullptr ? set.s[0] : s) || (rng_bits != 32 && rng_bits != 16)) return UQ_ERR_BAD_ARG;
    if (L->d > 0 && (g == nullptr || lev == nullptr || out == nullptr || !aligned(g, 16) || !aligned(lev, 16) ||
                     !aligned(out, 32) || !aligned(S_opt, 32)))
        return UQ_ERR_BAD_ARG;
    if (L->d > 0 && scales != nullptr && (idx == nullptr || !aligned(idx, 16))) return UQ_ERR_BAD_ARG;
    if (!uq::small_step_supported(*L, fmt)) return UQ_ERR_UNSUPPORTED;
    if (workspace == nullptr || !aligned(workspace, 8) || workspace_bytes < uq_workspace_bytes_small())
        return UQ_ERR_WORKSPACE;
    const cudaError_t e = scales != nullptr
        ? uq::launch_small_step_multi(*L, g, norm, set, idx_bits, seed, rng_bits, fmt, W, idx, lev, out, S_opt, status,
                                      workspace, (cudaStream_t)stream)
        : uq::launch_small_step(*L, g, norm, s, seed, rng_bits, fmt, W, lev, out, S_opt, status, workspace,
                                (cudaStream_t)stream);
    if (e == cudaErrorNotSupported) return UQ_ERR_UNSUPPORTED;
    return finish(e);
}

int uq_index_min(const uint8_t *rows, int R, int64_t row_bytes, int64_t nbytes, int idx_bits, uint8_t *idx, void *stream)
{
    if (R < 1 || R > UQ_MAX_WORKERS || nbytes < 0 || (nbytes & 3) != 0 || row_bytes < nbytes || (row_bytes & 3) != 0)
        return UQ_ERR_BAD_ARG;
    if (!idx_bits_ok(idx_bits)) return UQ_ERR_BAD_ARG;
    if (nbytes > 0 && (rows == nullptr || idx == nullptr || !aligned(rows, 4) || !aligned(idx, 4))) return UQ_ERR_BAD_ARG;
    return finish(uq::launch_index_min(rows, R, row_bytes, nbytes, idx_bits, idx, (cudaStream_t)stream));
}

int uq_randk_gather(const uq_layout *L, const void *g, int64_t K, uint64_t seed, int64_t *sel, void *gk,
                    int64_t gk_stride, uint32_t *status, void *stream)
{
    if (L == nullptr) return UQ_ERR_BAD_ARG;
    uq_layout dense = *L;                         // segments do not apply to the K-vector
    dense.seg_off = nullptr;
    dense.nseg = 1;
    dense.worker0 = 0;
    dense.coord0 = 0;
    if (!layout_ok(&dense) || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (K < 0 || K > dense.d || gk_stride < K || (gk_stride & 31) != 0) return UQ_ERR_BAD_ARG;
    if (gk_stride > 0 && (gk == nullptr || !aligned(gk, 16))) return UQ_ERR_BAD_ARG;
    if (K > 0 && (g == nullptr || sel == nullptr || !aligned(g, 16) || !aligned(sel, 8))) return UQ_ERR_BAD_ARG;
    return finish(uq::launch_randk_gather(dense, g, K, seed, sel, gk, gk_stride, status, (cudaStream_t)stream));
}

static int randk_scatter_common(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *dst, bool update,
                                float lr, uint32_t *status, void *stream)
{
    if (d < 0 || d > (int64_t)1 << 40 || K < 0 || K > d || !aligned(status, 4)) return UQ_ERR_BAD_ARG;
    if (K > 0 && (sel == nullptr || dst == nullptr || !aligned(sel, 8) || !aligned(dst, 4))) return UQ_ERR_BAD_ARG;
    if (!aligned(vals, 4) || (update && (vals == nullptr && K > 0)) || !(lr == lr)) return UQ_ERR_BAD_ARG;
    return finish(uq::launch_randk_scatter(d, K, sel, vals, dst, update, lr, status, (cudaStream_t)stream));
}

int uq_randk_scatter(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *out, uint32_t *status,
                     void *stream)
{
    return randk_scatter_common(d, K, sel, vals, out, false, 0.0f, status, stream);
}

int uq_randk_update(int64_t d, int64_t K, const int64_t *sel, const float *vals, float *theta, float lr,
                    uint32_t *status, void *stream)
{
    return randk_scatter_common(d, K, sel, vals, theta, true, lr, status, stream);
}

}  // extern "C"
