"""ctypes front end of the CPU oracle (``uq_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The CUDA package never imports this module.

Every function here only marshals numpy arrays into the C routine of the same name; all of the
method's arithmetic lives in the C file, which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "uq_oracle.c"
_LIB = _HERE / "libuq_oracle.so"

F32, BF16 = 0, 1
NORM_LINF, NORM_L2 = 0, 2

_CFLAGS = ["-std=c99", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-Wall"]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fused multiply-add, so every operator is one IEEE step)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(["gcc", *_CFLAGS, "-o", str(tmp), str(_SRC), "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
        _lib.uqo_draw.restype = C.c_uint32
        _lib.uqo_draw.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_int]
        _lib.uqo_get_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_of(g: np.ndarray) -> int:
    if g.dtype == np.float32:
        return F32
    if g.dtype == np.uint16:  # bfloat16 bit patterns
        return BF16
    raise TypeError(f"gradients must be float32 or uint16 (bf16 bits), got {g.dtype}")


def _seg(seg_off):
    if seg_off is None:
        return 1, None
    seg_off = np.ascontiguousarray(seg_off, dtype=np.int64)
    return len(seg_off) - 1, seg_off


def _check_g(g):
    """(M, d, row stride in elements) of a 2-D array whose rows are contiguous."""
    assert g.ndim == 2 and g.strides[1] == g.itemsize and g.strides[0] % g.itemsize == 0
    stride = g.strides[0] // g.itemsize if g.shape[0] > 1 else max(g.shape[1], 1)
    assert stride >= g.shape[1]
    return g.shape[0], g.shape[1], stride


def _rows(M, d, stride, dtype):
    """A zeroed [M, d] view with the given row stride (the C routines use one stride for all)."""
    return np.zeros((M, stride), dtype=dtype)[:, :d]


def _inject(h_inject, g, stride):
    """Injected draws laid out with the same row stride as g."""
    if h_inject is None:
        return None
    h_inject = np.asarray(h_inject, dtype=np.uint32)
    assert h_inject.shape == g.shape
    buf = _rows(g.shape[0], g.shape[1], stride, np.uint32)
    buf[...] = h_inject
    return buf


def set_threads(n: int) -> None:
    lib().uqo_set_threads(C.c_int(n))


def get_threads() -> int:
    return lib().uqo_get_threads()


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = np.asarray(ctr, dtype=np.uint32)
    key = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().uqo_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def draw(seed: int, m: int, i: int, rng_bits: int) -> int:
    return int(lib().uqo_draw(seed, m, i, rng_bits))


def agree_scale(g: np.ndarray, seg_off=None, norm: int = NORM_L2) -> np.ndarray:
    """W[j] = max over workers of the norm of segment j.  g is [M, d] (row stride d)."""
    M, d, stride = _check_g(g)
    nseg, so = _seg(seg_off)
    W = np.zeros(nseg, dtype=np.float32)
    lib().uqo_agree_scale(_p(g), _dtype_of(g), M, C.c_int64(d), C.c_int64(stride), nseg, _p(so),
                          norm, _p(W))
    return W


def encode_single(g, W, s, seed, rng_bits=32, seg_off=None, coord0=0, h_inject=None, worker0=0):
    """Levels zeta[m, i] (int8) of every worker; g holds coordinates coord0.. of each worker."""
    M, d, stride = _check_g(g)
    nseg, so = _seg(seg_off)
    W = np.ascontiguousarray(W, dtype=np.float32)
    assert W.size == nseg
    h_inject = _inject(h_inject, g, stride)
    lev = _rows(M, d, stride, np.int8)
    lib().uqo_encode_single(_p(g), _dtype_of(g), M, C.c_int64(coord0), C.c_int64(d),
                            C.c_int64(stride), nseg, _p(so), _p(W), C.c_int32(s), C.c_uint64(seed),
                            rng_bits, _p(h_inject), _p(lev), worker0)
    return lev


def select_scale_multi(g, W, scales, seg_off=None, coord0=0, return_own=False):
    """Shared scale index per coordinate (uint8, unpacked); optionally each worker's own index."""
    M, d, stride = _check_g(g)
    nseg, so = _seg(seg_off)
    W = np.ascontiguousarray(W, dtype=np.float32)
    assert W.size == nseg
    scales = np.ascontiguousarray(scales, dtype=np.int32)
    idx = np.zeros(d, dtype=np.uint8)
    own = _rows(M, d, stride, np.uint8) if return_own else None
    lib().uqo_select_scale_multi(_p(g), _dtype_of(g), M, C.c_int64(coord0), C.c_int64(d),
                                 C.c_int64(stride), nseg, _p(so), _p(W), _p(scales), len(scales),
                                 _p(idx), _p(own))
    return (idx, own) if return_own else idx


def encode_multi(g, W, scales, idx, seed, rng_bits=32, seg_off=None, coord0=0, h_inject=None, worker0=0):
    M, d, stride = _check_g(g)
    nseg, so = _seg(seg_off)
    W = np.ascontiguousarray(W, dtype=np.float32)
    assert W.size == nseg
    scales = np.ascontiguousarray(scales, dtype=np.int32)
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    assert idx.shape == (d,)
    h_inject = _inject(h_inject, g, stride)
    lev = _rows(M, d, stride, np.int8)
    lib().uqo_encode_multi(_p(g), _dtype_of(g), M, C.c_int64(coord0), C.c_int64(d),
                           C.c_int64(stride),
                           nseg, _p(so), _p(W), _p(scales), len(scales), _p(idx),
                           C.c_uint64(seed), rng_bits, _p(h_inject), _p(lev), worker0)
    return lev


def aggregate(lev: np.ndarray) -> np.ndarray:
    """S[i] = sum over workers of the int8 levels, in int32."""
    assert lev.dtype == np.int8
    M, d, stride = _check_g(lev)
    S = np.zeros(d, dtype=np.int32)
    lib().uqo_aggregate(_p(lev), M, C.c_int64(d), C.c_int64(stride), _p(S))
    return S


def decode(S, M, W, s=0, scales=None, idx=None, seg_off=None, coord0=0, f64=False):
    """Average gradient from the integer sums: W_j * S_i / (s_i * M)."""
    S = np.ascontiguousarray(S, dtype=np.int32)
    d = S.size
    nseg, so = _seg(seg_off)
    W = np.ascontiguousarray(W, dtype=np.float32)
    assert W.size == nseg
    if scales is not None:
        scales = np.ascontiguousarray(scales, dtype=np.int32)
        idx = np.ascontiguousarray(idx, dtype=np.uint8)
        assert idx.shape == (d,)
    out = np.zeros(d, dtype=np.float64 if f64 else np.float32)
    fn = lib().uqo_decode_f64 if f64 else lib().uqo_decode
    fn(_p(S), M, C.c_int64(coord0), C.c_int64(d), nseg, _p(so), _p(W), C.c_int32(s),
       _p(scales), _p(idx), _p(out))
    return out


def pack_levels_i4(lev: np.ndarray) -> np.ndarray:
    """Two 4-bit two's-complement levels per byte (row stride must be even)."""
    assert lev.dtype == np.int8
    M, d, stride = _check_g(lev)
    if M == 1:
        stride += stride & 1                 # a single row has no stride to respect
    assert stride % 2 == 0, "the row stride must be even"
    packed = np.zeros((M, stride // 2), dtype=np.uint8)
    lib().uqo_pack_levels_i4(_p(lev), M, C.c_int64(d), C.c_int64(stride), _p(packed))
    return packed[:, : (d + 1) // 2]


def pack_levels_i2(lev: np.ndarray) -> np.ndarray:
    """Four 2-bit two's-complement levels per byte (row stride must be a multiple of 4)."""
    assert lev.dtype == np.int8
    M, d, stride = _check_g(lev)
    if M == 1:
        stride = -(-stride // 4) * 4
    assert stride % 4 == 0, "the row stride must be a multiple of 4"
    packed = np.zeros((M, stride // 4), dtype=np.uint8)
    lib().uqo_pack_levels_i2(_p(lev), M, C.c_int64(d), C.c_int64(stride), _p(packed))
    return packed[:, : (d + 3) // 4]


def pack_levels_i6p(lev: np.ndarray, stride: int) -> np.ndarray:
    """6-bit levels in two planes per row ([M, row_bytes]: nibbles of bits 0..3 in the first
    stride/2 bytes, 2-bit fields of bits 4..5 after them); stride = the layout's row stride in
    coordinates (a multiple of 32), rows are 3*stride/4 bytes rounded up to 16."""
    assert lev.dtype == np.int8 and stride % 32 == 0
    M, d, lev_stride = _check_g(lev)
    row_bytes = (stride // 2 + stride // 4 + 15) // 16 * 16
    packed = np.zeros((M, row_bytes), dtype=np.uint8)
    lib().uqo_pack_levels_i6p(_p(lev), M, C.c_int64(d), C.c_int64(lev_stride), C.c_int64(stride), C.c_int64(row_bytes),
                              _p(packed))
    return packed


def index_min(rows: np.ndarray) -> np.ndarray:
    """Minimum over the rows of an [R, d] array of (unpacked) scale indices."""
    rows = np.ascontiguousarray(rows, dtype=np.uint8)
    R, d = rows.shape
    idx = np.zeros(d, dtype=np.uint8)
    lib().uqo_index_min(_p(rows), R, C.c_int64(d), _p(idx))
    return idx


def pack_index(idx: np.ndarray, idx_bits: int) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    per = 8 // idx_bits
    packed = np.zeros((idx.size + per - 1) // per, dtype=np.uint8)
    lib().uqo_pack_index(_p(idx), C.c_int64(idx.size), idx_bits, _p(packed))
    return packed


def sgd_update(g_hat, theta, mom=None, lr=0.1, mu=0.0, wd=0.0):
    """theta (and the momentum buffer) after one step; inputs are not modified."""
    g_hat = np.ascontiguousarray(g_hat, dtype=np.float32)
    theta = np.array(theta, dtype=np.float32, copy=True)
    mom = None if mom is None else np.array(mom, dtype=np.float32, copy=True)
    assert theta.shape == g_hat.shape and (mom is None or mom.shape == g_hat.shape)
    lib().uqo_sgd_update(_p(g_hat), C.c_int64(g_hat.size), _p(theta), _p(mom), C.c_float(lr), C.c_float(mu),
                         C.c_float(wd))
    return theta, mom


# ---------------------------------------------------------------------------------------------
# GlobalRandK (Sections "GlobalRandKMaxNorm Compression", "GlobalRandKMaxNormMultiScale Compression")
# ---------------------------------------------------------------------------------------------

def randk_indices(d: int, K: int, seed: int) -> np.ndarray:
    """The K distinct coordinates every worker keeps at this seed, in selection order."""
    assert 0 <= K <= d
    sel = np.zeros(K, dtype=np.int64)
    lib().uqo_randk_indices(C.c_int64(d), C.c_int64(K), C.c_uint64(seed), _p(sel))
    return sel


def randk_gather(g: np.ndarray, sel: np.ndarray) -> np.ndarray:
    """[M, K] view (row stride = K rounded up to 32) of the chosen coordinates of every worker."""
    M, d, stride = _check_g(g)
    sel = np.ascontiguousarray(sel, dtype=np.int64)
    K = sel.size
    strideK = max(32, -(-K // 32) * 32)
    gk = np.zeros((M, strideK), dtype=g.dtype)
    lib().uqo_randk_gather(_p(g), _dtype_of(g), M, C.c_int64(stride), C.c_int64(K), _p(sel), _p(gk),
                           C.c_int64(strideK))
    return gk[:, :K]


def randk_scatter(sel: np.ndarray, vals, out: np.ndarray) -> np.ndarray:
    """out with out[sel[t]] = vals[t] (vals None: 0); modifies and returns out (float32)."""
    sel = np.ascontiguousarray(sel, dtype=np.int64)
    assert out.dtype == np.float32 and out.flags.c_contiguous
    vals = None if vals is None else np.ascontiguousarray(vals, dtype=np.float32)
    lib().uqo_randk_scatter(C.c_int64(sel.size), _p(sel), _p(vals), _p(out))
    return out


def randk_update(sel: np.ndarray, vals: np.ndarray, theta: np.ndarray, lr: float) -> np.ndarray:
    """A copy of theta after theta[sel] -= lr * vals."""
    sel = np.ascontiguousarray(sel, dtype=np.int64)
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    theta = np.array(theta, dtype=np.float32, copy=True)
    lib().uqo_randk_update(C.c_int64(sel.size), _p(sel), _p(vals), _p(theta), C.c_float(lr))
    return theta
