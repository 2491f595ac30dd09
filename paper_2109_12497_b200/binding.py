"""Thin ctypes binding of the C ABI in ``include/uq.h``.

Argument marshalling only: every function takes torch CUDA tensors (device memory and the
current stream are torch's), checks shapes and dtypes, and calls the C entry point of the same
name.  All arithmetic runs in the CUDA kernels of ``libuq_b200.so``; there is no CPU path, and
a missing or unloadable library is an error.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Optional, Sequence

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libuq_b200.so"

UQ_OK, UQ_ERR_BAD_ARG, UQ_ERR_CUDA, UQ_ERR_UNSUPPORTED, UQ_ERR_WORKSPACE = range(5)
UQ_F32, UQ_BF16 = 0, 1
UQ_NORM_LINF, UQ_NORM_L2 = 0, 2
UQ_FMT_I8, UQ_FMT_I4X2, UQ_FMT_I2X4, UQ_FMT_I6P = 0, 1, 2, 3
UQ_SRC_LEVELS, UQ_SRC_SUMS = 0, 1
UQ_STATUS_NONFINITE, UQ_STATUS_BAD_SEGMENTS, UQ_STATUS_SCALE_OVERFLOW, UQ_STATUS_BAD_INDEX = 1, 2, 4, 8
UQ_STATUS_TIMEOUT = 16

EXPORTS = (
    "uq_version", "uq_last_cuda_error", "uq_error_string", "uq_workspace_bytes", "uq_index_bytes",
    "uq_workspace_bytes_small",
    "uq_agree_scale", "uq_agree_scale_static", "uq_encode_single", "uq_select_scale_multi", "uq_encode_multi",
    "uq_aggregate", "uq_decode", "uq_decode_update", "uq_randk_gather", "uq_randk_scatter", "uq_randk_update", "uq_index_min", "uq_decode_rows", "uq_select_encode_multi", "uq_encode_decode", "uq_select_encode_decode_multi", "uq_step",
    "uq_step_small",
)


class uq_layout(C.Structure):
    _fields_ = [
        ("d", C.c_int64),
        ("worker_stride", C.c_int64),
        ("seg_off", C.c_void_p),
        ("M", C.c_int32),
        ("nseg", C.c_int32),
        ("dtype", C.c_int32),
        ("worker0", C.c_int32),
        ("coord0", C.c_int64),
    ]


class UqError(RuntimeError):
    def __init__(self, fn: str, code: int):
        msg = lib().uq_error_string(code).decode()
        if code == UQ_ERR_CUDA:
            msg += f" [cuda error {lib().uq_last_cuda_error()}]"
        super().__init__(f"{fn}: {msg} (code {code})")
        self.code = code


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """The loaded CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2109_12497_b200.build` "
                "(the quantizer has no CPU fallback)")
        L = C.CDLL(str(LIB_PATH))
        P, I, U64, SZ = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
        LP = C.POINTER(uq_layout)
        L.uq_version.restype = I
        L.uq_last_cuda_error.restype = I
        L.uq_error_string.restype = C.c_char_p
        L.uq_error_string.argtypes = [I]
        L.uq_workspace_bytes.restype = SZ
        L.uq_workspace_bytes.argtypes = [LP]
        L.uq_index_bytes.restype = SZ
        L.uq_index_bytes.argtypes = [LP, I]
        L.uq_agree_scale.argtypes = [LP, P, I, P, P, P, SZ, P]
        L.uq_step.argtypes = [LP, P, I, I, P, I, I, U64, I, I, P, P, P, P, P, P, P, SZ, P]
        L.uq_step_small.argtypes = [LP, P, I, I, P, I, I, U64, I, I, P, P, P, P, P, P, P, SZ, P]
        L.uq_workspace_bytes_small.restype = SZ
        L.uq_workspace_bytes_small.argtypes = []
        L.uq_agree_scale_static.argtypes = [LP, P, I, P, P, P]
        L.uq_encode_single.argtypes = [LP, P, P, I, U64, I, I, P, P, P]
        L.uq_select_scale_multi.argtypes = [LP, P, P, P, I, I, P, P, P]
        L.uq_encode_multi.argtypes = [LP, P, P, P, I, P, I, U64, I, I, P, P, P]
        L.uq_aggregate.argtypes = [LP, P, I, P, P]
        L.uq_decode.argtypes = [LP, P, I, I, P, I, P, I, P, I, P, P, P]
        F = C.c_float
        L.uq_decode_update.argtypes = [LP, P, I, P, I, P, I, P, I, P, P, F, F, F, P, P]
        I64 = C.c_int64
        L.uq_select_encode_multi.argtypes = [LP, P, P, P, I, I, U64, I, I, P, P, P, P]
        L.uq_decode_rows.argtypes = [LP, P, I, P, I, P, I, P, I, P, P, P]
        L.uq_encode_decode.argtypes = [LP, P, P, I, P, I, P, I, U64, I, I, P, P, P, P]
        L.uq_select_encode_decode_multi.argtypes = [LP, P, P, P, I, I, U64, I, I, P, P, P, P, P]
        L.uq_index_min.argtypes = [P, I, I64, I64, I, P, P]
        L.uq_randk_gather.argtypes = [LP, P, I64, U64, P, P, I64, P, P]
        L.uq_randk_scatter.argtypes = [I64, I64, P, P, P, P, P]
        L.uq_randk_update.argtypes = [I64, I64, P, P, P, F, P, P]
        for name in EXPORTS[7:]:
            getattr(L, name).restype = I
        _lib = L
    return _lib


def require_current_device(index: Optional[int], current: int, what: str = "tensor") -> None:
    """Every call launches on the CURRENT device's current stream, so a tensor on another device
    would hand that device a pointer it cannot use (a fault, or silent peer traffic): refuse."""
    if index is None or index != current:
        raise ValueError(f"uq: {what} lives on CUDA device {index}, but the current device is {current}; "
                         f"make its device current first (torch.cuda.device / set_device)")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("uq: tensors must live on a CUDA device")
    require_current_device(t.device.index, torch.cuda.current_device())
    return t.data_ptr()


def _stream() -> int:
    """The raw handle of the current stream of the current CUDA device."""
    return torch._C._cuda_getCurrentRawStream(torch.cuda.current_device())


def _check(fn: str, code: int) -> None:
    if code != UQ_OK:
        raise UqError(fn, code)


def _scales(scales: Sequence[int]):
    arr = (C.c_int32 * len(scales))(*[int(s) for s in scales])
    return arr, len(scales)


class Layout:
    """Shape of the M workers' gradient buffers: d coordinates per worker in rows of
    ``worker_stride`` coordinates, cut into segments that each share one scale."""

    def __init__(self, M: int, d: int, worker_stride: int, dtype: torch.dtype,
                 seg_off: Optional[torch.Tensor] = None, worker0: int = 0, coord0: int = 0):
        if dtype not in (torch.float32, torch.bfloat16):
            raise ValueError("uq: gradients are float32 or bfloat16")
        if seg_off is not None:
            if seg_off.dtype != torch.int64 or not seg_off.is_cuda or seg_off.dim() != 1:
                raise ValueError("uq: seg_off is a 1-D int64 CUDA tensor")
            seg_off = seg_off.contiguous()
        self.M, self.d, self.worker_stride, self.dtype, self.seg_off = M, d, worker_stride, dtype, seg_off
        self.nseg = 1 if seg_off is None else seg_off.numel() - 1
        self.worker0, self.coord0 = worker0, coord0
        self.c = uq_layout(d, worker_stride, _ptr(seg_off), M, self.nseg,
                           UQ_F32 if dtype == torch.float32 else UQ_BF16, worker0, coord0)

    def ref(self):
        return C.byref(self.c)

    def workspace_bytes(self) -> int:
        return int(lib().uq_workspace_bytes(self.ref()))


    def index_bytes(self, idx_bits: int) -> int:
        return int(lib().uq_index_bytes(self.ref(), idx_bits))

    def level_row_bytes(self, fmt: int) -> int:
        if fmt == UQ_FMT_I6P:                       # a nibble plane and a 2-bit plane, rows rounded up to 16 bytes
            return (self.worker_stride // 2 + self.worker_stride // 4 + 15) // 16 * 16
        return self.worker_stride >> fmt            # 1, 2 or 4 coordinates per byte

    def check_g(self, g: torch.Tensor) -> None:
        if g.dtype != self.dtype or g.dim() != 2 or g.shape[0] != self.M or g.shape[1] != self.worker_stride \
                or not g.is_contiguous():
            raise ValueError(f"uq: g must be a contiguous [{self.M}, {self.worker_stride}] {self.dtype} tensor")

    def check_lev(self, lev: torch.Tensor, fmt: int) -> None:
        if lev.dtype not in (torch.int8, torch.uint8) or lev.dim() != 2 or lev.shape[0] != self.M \
                or lev.shape[1] != self.level_row_bytes(fmt) or not lev.is_contiguous():
            raise ValueError(f"uq: lev must be a contiguous [{self.M}, {self.level_row_bytes(fmt)}] byte tensor")

    def check_vec(self, t: torch.Tensor, dtype: torch.dtype, n: int, what: str) -> None:
        if t.dtype != dtype or t.dim() != 1 or t.numel() < n or not t.is_contiguous():
            raise ValueError(f"uq: {what} must be a contiguous 1-D {dtype} tensor with >= {n} elements")


def uq_version() -> int:
    return int(lib().uq_version())


def uq_agree_scale(layout: Layout, g: torch.Tensor, norm: int, W: torch.Tensor,
                   status: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    layout.check_g(g)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    _check("uq_agree_scale", lib().uq_agree_scale(
        layout.ref(), _ptr(g), norm, _ptr(W), _ptr(status), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))


STATIC_SCRATCH_BYTES = 4 << 20


def uq_agree_scale_static(layout: Layout, g: torch.Tensor, norm: int, W: torch.Tensor,
                          status: Optional[torch.Tensor]) -> None:
    """uq_agree_scale without a workspace argument, for callers that cannot allocate one: the
    scratch is a 4 MiB array inside the library (layouts that need more raise UqError with
    UQ_ERR_WORKSPACE).  Calls on one device share that array, so keep them on one stream; the
    first call on a device does a one-time address lookup and belongs in set-up code."""
    layout.check_g(g)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    _check("uq_agree_scale_static", lib().uq_agree_scale_static(
        layout.ref(), _ptr(g), norm, _ptr(W), _ptr(status), _stream()))


def uq_encode_single(layout: Layout, g: torch.Tensor, W: torch.Tensor, s: int, seed: int, rng_bits: int,
                     fmt: int, lev: torch.Tensor, status: Optional[torch.Tensor]) -> None:
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    _check("uq_encode_single", lib().uq_encode_single(
        layout.ref(), _ptr(g), _ptr(W), s, seed, rng_bits, fmt, _ptr(lev), _ptr(status), _stream()))


def uq_select_scale_multi(layout: Layout, g: torch.Tensor, W: torch.Tensor, scales: Sequence[int],
                          idx_bits: int, idx: torch.Tensor, status: Optional[torch.Tensor]) -> None:
    layout.check_g(g)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    arr, N = _scales(scales)
    _check("uq_select_scale_multi", lib().uq_select_scale_multi(
        layout.ref(), _ptr(g), _ptr(W), arr, N, idx_bits, _ptr(idx), _ptr(status), _stream()))


def uq_encode_multi(layout: Layout, g: torch.Tensor, W: torch.Tensor, scales: Sequence[int],
                    idx: torch.Tensor, idx_bits: int, seed: int, rng_bits: int, fmt: int,
                    lev: torch.Tensor, status: Optional[torch.Tensor]) -> None:
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    arr, N = _scales(scales)
    _check("uq_encode_multi", lib().uq_encode_multi(
        layout.ref(), _ptr(g), _ptr(W), arr, N, _ptr(idx), idx_bits, seed, rng_bits, fmt, _ptr(lev),
        _ptr(status), _stream()))


def uq_aggregate(layout: Layout, lev: torch.Tensor, fmt: int, S: torch.Tensor) -> None:
    layout.check_lev(lev, fmt)
    layout.check_vec(S, torch.int32, layout.d, "S")
    _check("uq_aggregate", lib().uq_aggregate(layout.ref(), _ptr(lev), fmt, _ptr(S), _stream()))


def uq_decode(layout: Layout, src: torch.Tensor, src_kind: int, fmt: int, W: torch.Tensor, s: int,
              scales: Optional[Sequence[int]], idx: Optional[torch.Tensor], idx_bits: int,
              out: torch.Tensor, S_opt: Optional[torch.Tensor] = None) -> None:
    if src_kind == UQ_SRC_LEVELS:
        layout.check_lev(src, fmt)
    else:
        layout.check_vec(src, torch.int32, layout.d, "src")
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    if S_opt is not None:
        layout.check_vec(S_opt, torch.int32, layout.d, "S_opt")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    _check("uq_decode", lib().uq_decode(
        layout.ref(), _ptr(src), src_kind, fmt, _ptr(W), s, arr, N, _ptr(idx) if scales is not None else None,
        idx_bits, _ptr(out), _ptr(S_opt), _stream()))


def uq_decode_update(layout: Layout, lev: torch.Tensor, fmt: int, W: torch.Tensor, s: int,
                     scales: Optional[Sequence[int]], idx: Optional[torch.Tensor], idx_bits: int,
                     theta: torch.Tensor, momentum: Optional[torch.Tensor], lr: float, mu: float = 0.0,
                     wd: float = 0.0, out: Optional[torch.Tensor] = None) -> None:
    """Sum of the level rows, reconstruction and the SGD step on theta (and the momentum buffer)
    in one kernel; ``out`` optionally also receives the reconstructed gradient."""
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(theta, torch.float32, layout.d, "theta")
    if momentum is not None:
        layout.check_vec(momentum, torch.float32, layout.d, "momentum")
    if out is not None:
        layout.check_vec(out, torch.float32, layout.d, "out")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    _check("uq_decode_update", lib().uq_decode_update(
        layout.ref(), _ptr(lev), fmt, _ptr(W), s, arr, N, _ptr(idx) if scales is not None else None, idx_bits,
        _ptr(theta), _ptr(momentum), lr, mu, wd, _ptr(out), _stream()))


def uq_randk_gather(layout: Layout, g: torch.Tensor, K: int, seed: int, sel: torch.Tensor, gk: torch.Tensor,
                    status: Optional[torch.Tensor] = None) -> None:
    """The K coordinates all workers keep at this seed (sel, int64 [K]) and their values
    gk[m, t] = g[m, sel[t]] in a compact [M, gk_stride] buffer whose row padding is zeroed."""
    layout.check_g(g)
    if gk.dtype != layout.dtype or gk.dim() != 2 or gk.shape[0] != layout.M or not gk.is_contiguous():
        raise ValueError(f"uq: gk must be a contiguous [{layout.M}, gk_stride] {layout.dtype} tensor")
    layout.check_vec(sel, torch.int64, K, "sel")
    _check("uq_randk_gather", lib().uq_randk_gather(
        layout.ref(), _ptr(g), K, seed, _ptr(sel), _ptr(gk), gk.shape[1], _ptr(status), _stream()))


def _check_randk(d: int, K: int, sel: torch.Tensor, vals: Optional[torch.Tensor], dst: torch.Tensor, what: str):
    for t, dt, n, name in ((sel, torch.int64, K, "sel"), (vals, torch.float32, K, "vals"), (dst, torch.float32, d, what)):
        if t is not None and (t.dtype != dt or t.dim() != 1 or t.numel() < n or not t.is_contiguous()):
            raise ValueError(f"uq: {name} must be a contiguous 1-D {dt} tensor with >= {n} elements")


def uq_randk_scatter(d: int, K: int, sel: torch.Tensor, vals: Optional[torch.Tensor], out: torch.Tensor,
                     status: Optional[torch.Tensor] = None) -> None:
    """out[sel[t]] = vals[t] (vals None: 0); the other coordinates of out are left alone."""
    _check_randk(d, K, sel, vals, out, "out")
    _check("uq_randk_scatter", lib().uq_randk_scatter(d, K, _ptr(sel), _ptr(vals), _ptr(out), _ptr(status),
                                                      _stream()))


def uq_randk_update(d: int, K: int, sel: torch.Tensor, vals: torch.Tensor, theta: torch.Tensor, lr: float,
                    status: Optional[torch.Tensor] = None) -> None:
    """theta[sel[t]] -= lr * vals[t]."""
    _check_randk(d, K, sel, vals, theta, "theta")
    _check("uq_randk_update", lib().uq_randk_update(d, K, _ptr(sel), _ptr(vals), _ptr(theta), lr, _ptr(status),
                                                    _stream()))


def uq_index_min(rows: torch.Tensor, idx_bits: int, idx: torch.Tensor, nbytes: Optional[int] = None) -> None:
    """Field-wise minimum over the rows of a [R, row_bytes] uint8 tensor of packed scale indices
    (one row per process) into idx; nbytes defaults to the whole row."""
    if rows.dtype != torch.uint8 or rows.dim() != 2 or not rows.is_contiguous():
        raise ValueError("uq: rows must be a contiguous [R, row_bytes] uint8 tensor")
    nbytes = rows.shape[1] if nbytes is None else nbytes
    if idx.dtype != torch.uint8 or idx.dim() != 1 or idx.numel() < nbytes or not idx.is_contiguous():
        raise ValueError(f"uq: idx must be a contiguous uint8 tensor with >= {nbytes} elements")
    _check("uq_index_min", lib().uq_index_min(_ptr(rows), rows.shape[0], rows.shape[1], nbytes, idx_bits, _ptr(idx),
                                              _stream()))


def uq_decode_rows(layout: Layout, lev_rows: Sequence[int], fmt: int, W: torch.Tensor, s: int,
                   scales: Optional[Sequence[int]], idx: Optional[torch.Tensor], idx_bits: int,
                   out: torch.Tensor, S_opt: Optional[torch.Tensor] = None) -> None:
    """uq_decode over level rows given as M device addresses (one per worker, in worker order);
    a row may live in a peer GPU's memory that is mapped into this process."""
    if len(lev_rows) != layout.M:
        raise ValueError(f"uq: lev_rows must hold {layout.M} addresses")
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    if S_opt is not None:
        layout.check_vec(S_opt, torch.int32, layout.d, "S_opt")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    rows = (C.c_void_p * layout.M)(*[int(a) for a in lev_rows])
    _check("uq_decode_rows", lib().uq_decode_rows(
        layout.ref(), rows, fmt, _ptr(W), s, arr, N, _ptr(idx) if scales is not None else None, idx_bits,
        _ptr(out), _ptr(S_opt), _stream()))


def uq_select_encode_multi(layout: Layout, g: torch.Tensor, W: torch.Tensor, scales: Sequence[int], idx_bits: int,
                           seed: int, rng_bits: int, fmt: int, idx: torch.Tensor, lev: torch.Tensor,
                           status: Optional[torch.Tensor]) -> None:
    """uq_select_scale_multi + uq_encode_multi in one kernel (all workers in this buffer)."""
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    arr, N = _scales(scales)
    _check("uq_select_encode_multi", lib().uq_select_encode_multi(
        layout.ref(), _ptr(g), _ptr(W), arr, N, idx_bits, seed, rng_bits, fmt, _ptr(idx), _ptr(lev), _ptr(status),
        _stream()))



def uq_select_encode_decode_multi(layout: Layout, g: torch.Tensor, W: torch.Tensor, scales: Sequence[int], idx_bits: int,
                                  seed: int, rng_bits: int, fmt: int, idx: torch.Tensor, lev: torch.Tensor,
                                  out: torch.Tensor, status: Optional[torch.Tensor]) -> None:
    """uq_select_encode_multi + uq_decode(levels) as one call (one kernel where uq_encode_decode is one)."""
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    arr, N = _scales(scales)
    _check("uq_select_encode_decode_multi", lib().uq_select_encode_decode_multi(
        layout.ref(), _ptr(g), _ptr(W), arr, N, idx_bits, seed, rng_bits, fmt, _ptr(idx), _ptr(lev), _ptr(out),
        _ptr(status), _stream()))


def uq_encode_decode(layout: Layout, g: torch.Tensor, W: torch.Tensor, s: int, scales: Optional[Sequence[int]],
                     idx: Optional[torch.Tensor], idx_bits: int, seed: int, rng_bits: int, fmt: int, lev: torch.Tensor,
                     out: torch.Tensor, status: Optional[torch.Tensor]) -> None:
    """uq_encode_single / uq_encode_multi + uq_decode(levels) as one call (one kernel for int8 levels, 16-bit draws and M <= 8)."""
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    _check("uq_encode_decode", lib().uq_encode_decode(
        layout.ref(), _ptr(g), _ptr(W), s, arr, N, _ptr(idx) if scales is not None else None, idx_bits, seed, rng_bits,
        fmt, _ptr(lev), _ptr(out), _ptr(status), _stream()))


def uq_step(layout: Layout, g: torch.Tensor, norm: int, s: int, scales: Optional[Sequence[int]], idx_bits: int,
            seed: int, rng_bits: int, fmt: int, W: torch.Tensor, idx: Optional[torch.Tensor], lev: torch.Tensor,
            out: torch.Tensor, S_opt: Optional[torch.Tensor], status: Optional[torch.Tensor],
            workspace: torch.Tensor) -> None:
    """One whole step (agree-scale, [select], encode, aggregate + reconstruct) in one call."""
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, layout.nseg, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    if S_opt is not None:
        layout.check_vec(S_opt, torch.int32, layout.d, "S_opt")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    _check("uq_step", lib().uq_step(
        layout.ref(), _ptr(g), norm, s, arr, N, idx_bits, seed, rng_bits, fmt, _ptr(W),
        _ptr(idx) if scales is not None else None, _ptr(lev), _ptr(out), _ptr(S_opt), _ptr(status), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))


SMALL_STEP_MAX_WORKERS = 8


def uq_workspace_bytes_small() -> int:
    return int(lib().uq_workspace_bytes_small())


def small_step_supported(layout: Layout, fmt: int) -> bool:
    """Whether uq_step_small takes this configuration (one segment, M <= 8, one-plane levels)."""
    return layout.nseg == 1 and layout.M <= SMALL_STEP_MAX_WORKERS and fmt in (UQ_FMT_I8, UQ_FMT_I4X2, UQ_FMT_I2X4)


def uq_step_small(layout: Layout, g: torch.Tensor, norm: int, s: int, scales: Optional[Sequence[int]], idx_bits: int,
                  seed: int, rng_bits: int, fmt: int, W: torch.Tensor, idx: Optional[torch.Tensor], lev: torch.Tensor,
                  out: torch.Tensor, S_opt: Optional[torch.Tensor], status: Optional[torch.Tensor],
                  workspace: torch.Tensor) -> None:
    """The whole step of either quantizer as one cooperative kernel (small gradients); arguments as
    uq_step.  ``workspace``: zero-filled before its first use (the kernel leaves its counters
    zero), one call at a time."""
    layout.check_g(g)
    layout.check_lev(lev, fmt)
    layout.check_vec(W, torch.float32, 1, "W")
    layout.check_vec(out, torch.float32, layout.d, "out")
    if S_opt is not None:
        layout.check_vec(S_opt, torch.int32, layout.d, "S_opt")
    arr, N = (None, 0)
    if scales is not None:
        arr, N = _scales(scales)
        layout.check_vec(idx, torch.uint8, layout.index_bytes(idx_bits), "idx")
    _check("uq_step_small", lib().uq_step_small(
        layout.ref(), _ptr(g), norm, s, arr, N, idx_bits, seed, rng_bits, fmt, _ptr(W),
        _ptr(idx) if scales is not None else None, _ptr(lev), _ptr(out), _ptr(S_opt), _ptr(status), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))
