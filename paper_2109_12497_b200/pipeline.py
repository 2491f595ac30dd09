"""One quantize -> aggregate -> reconstruct step over M resident worker buffers.

``Quantizer`` owns the device buffers of one configuration (scales, scale indices, levels,
scratch, output) and enqueues the C-ABI calls of Algorithm 1 (single-scale) or Algorithm 2
(multi-scale) in order on the current stream.  It holds no arithmetic: each stage is one call
into the CUDA library.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as B


ONE_KERNEL_MAX_BYTES = 8 << 20      # gradients of all workers up to this size take the one-kernel step


class Quantizer:
    def __init__(self, M: int, d: int, dtype: torch.dtype = torch.float32,
                 seg_off: Optional[Sequence[int]] = None, s: int = 127,
                 scales: Optional[Sequence[int]] = None, fmt: int = B.UQ_FMT_I8, idx_bits: int = 0,
                 norm: int = B.UQ_NORM_L2, rng_bits: int = 32, keep_sums: bool = False,
                 device: str | torch.device = "cuda", fused_select: Optional[bool] = None,
                 one_kernel: Optional[bool] = None):
        B.lib()                                     # fail now if the CUDA library is not built
        dev = torch.device(device)
        if dev.type == "cuda" and dev.index is None:
            dev = torch.device("cuda", torch.cuda.current_device())
        self.device = dev
        self.M, self.d, self.dtype = M, d, dtype
        self.stride = -(-d // 32) * 32
        self.multi = scales is not None and idx_bits != 0
        # multi-scale: whether selection + sharing run inside the encoder's kernel (one kernel for M <= 8,
        # the gradients read once, same bits) instead of as a streaming kernel of their own.  None = the
        # library's own choice (uq_step: inside where the encoder also aggregates and reconstructs, i.e.
        # int8 levels, 16-bit draws, M <= 8 and no integer sums kept; a kernel of its own otherwise).
        self.fused_select = None if fused_select is None else bool(fused_select) and self.multi
        self.s = int(scales[0]) if self.multi else int(s)
        self.scales = [int(x) for x in scales] if self.multi else None
        self.fmt, self.idx_bits, self.norm, self.rng_bits = fmt, idx_bits if self.multi else 0, norm, rng_bits
        seg_dev = None
        if seg_off is not None and len(seg_off) > 2:
            seg_dev = torch.as_tensor(np.asarray(seg_off, dtype=np.int64), device=dev)
        self.layout = B.Layout(M, d, self.stride, dtype, seg_dev)
        nseg = self.layout.nseg
        self.W = torch.zeros(nseg, dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        # one segment, few workers, and so small that the step is bound by its launches: the whole step as one cooperative kernel (uq_step_small).  None = decide by size.
        fits = B.small_step_supported(self.layout, fmt)
        if one_kernel and not fits:
            raise ValueError("uq: the one-kernel step takes one segment, M <= 8 and one-plane level formats")
        self.one_kernel = fits and (one_kernel if one_kernel is not None
                                    else M * d * (4 if dtype == torch.float32 else 2) <= ONE_KERNEL_MAX_BYTES)
        self.workspace = torch.empty(max(8, self.layout.workspace_bytes()), dtype=torch.uint8, device=dev)
        # The one-kernel step keeps its barrier counters in the first bytes of its scratch, wants them
        # zero before the first call and leaves them zero: a buffer of its own, never handed to
        # uq_agree_scale (whose partial sums would overwrite the counters).
        self.small_workspace = (torch.zeros(max(8, B.uq_workspace_bytes_small()), dtype=torch.uint8, device=dev)
                                if self.one_kernel else None)
        self.lev = torch.empty((M, self.layout.level_row_bytes(fmt)), dtype=torch.int8, device=dev)
        self.idx = (torch.empty(max(16, self.layout.index_bytes(self.idx_bits)), dtype=torch.uint8, device=dev)
                    if self.multi else None)
        self.out = torch.empty(max(d, 1), dtype=torch.float32, device=dev)
        self.S = torch.empty(max(d, 1), dtype=torch.int32, device=dev) if keep_sums else None
        self._small_call = None
        self._step_call = None
        self._out_view = self.out[: self.d]

    # the four stages, each one C-ABI call -------------------------------------------------------
    def agree_scale(self, g: torch.Tensor) -> None:
        B.uq_agree_scale(self.layout, g, self.norm, self.W, self.status, self.workspace)

    def select_scale(self, g: torch.Tensor) -> None:
        B.uq_select_scale_multi(self.layout, g, self.W, self.scales, self.idx_bits, self.idx, self.status)

    def encode(self, g: torch.Tensor, seed: int) -> None:
        if self.multi:
            B.uq_encode_multi(self.layout, g, self.W, self.scales, self.idx, self.idx_bits, seed,
                              self.rng_bits, self.fmt, self.lev, self.status)
        else:
            B.uq_encode_single(self.layout, g, self.W, self.s, seed, self.rng_bits, self.fmt, self.lev,
                               self.status)

    def select_encode(self, g: torch.Tensor, seed: int) -> None:
        """Multi-scale: scale selection, scale sharing and quantization in one call."""
        B.uq_select_encode_multi(self.layout, g, self.W, self.scales, self.idx_bits, seed, self.rng_bits, self.fmt,
                                 self.idx, self.lev, self.status)

    def select_encode_decode(self, g: torch.Tensor, seed: int) -> None:
        """Multi-scale: everything behind the scale agreement in one call."""
        B.uq_select_encode_decode_multi(self.layout, g, self.W, self.scales, self.idx_bits, seed, self.rng_bits,
                                        self.fmt, self.idx, self.lev, self.out, self.status)

    def aggregate_decode(self) -> None:
        B.uq_decode(self.layout, self.lev, B.UQ_SRC_LEVELS, self.fmt, self.W, self.s, self.scales, self.idx,
                    self.idx_bits, self.out, self.S)

    def encode_decode(self, g: torch.Tensor, seed: int) -> None:
        """Quantization, integer aggregation and reconstruction as one call (what the step makes when
        the integer sums are not kept; one kernel for int8 levels, 16-bit draws and M <= 8)."""
        B.uq_encode_decode(self.layout, g, self.W, self.s, self.scales, self.idx, self.idx_bits, seed, self.rng_bits,
                           self.fmt, self.lev, self.out, self.status)

    @property
    def selects_inside(self) -> bool:
        """Multi-scale: whether the step's selection runs inside the encoder's kernel."""
        if not self.multi:
            return False
        return self.fused_decode if self.fused_select is None else self.fused_select

    @property
    def fused_decode(self) -> bool:
        """Whether the step's encoder also aggregates and reconstructs (uq_encode_decode as one kernel)."""
        return (self.S is None and self.fmt == B.UQ_FMT_I8 and self.layout.M <= B.SMALL_STEP_MAX_WORKERS
                and self.rng_bits == 16)

    def aggregate_decode_update(self, theta: torch.Tensor, momentum: Optional[torch.Tensor], lr: float,
                                mu: float = 0.0, wd: float = 0.0) -> None:
        """Fused aggregation, reconstruction and SGD step on theta (Algorithm 1/2, last three lines)."""
        B.uq_decode_update(self.layout, self.lev, self.fmt, self.W, self.s, self.scales, self.idx, self.idx_bits,
                           theta, momentum, lr, mu, wd)

    def step(self, g: torch.Tensor, seed: int = 0) -> torch.Tensor:
        """g: [M, stride] gradients of all workers -> the reconstructed average gradient [d]."""
        if self.one_kernel:
            # every buffer but g is this object's own: their addresses are marshalled once, not per
            # step (the checked wrapper B.uq_step_small costs about as much host time as the kernel runs)
            self._check_devices(g)
            if self._small_call is None:
                ptr = lambda t: None if t is None else t.data_ptr()
                arr, N = B._scales(self.scales) if self.multi else (None, 0)
                self._small_call = (B.lib().uq_step_small, self.layout.ref(), arr, N,
                                    (ptr(self.W), ptr(self.idx), ptr(self.lev), ptr(self.out), ptr(self.S),
                                     ptr(self.status), ptr(self.small_workspace), self.small_workspace.numel()))
            fn, ref, arr, N, tail = self._small_call
            rc = fn(ref, g.data_ptr(), self.norm, self.s, arr, N, self.idx_bits, seed, self.rng_bits, self.fmt, *tail,
                    B._stream())
            if rc != B.UQ_OK:
                raise B.UqError("uq_step_small", rc)
            return self._out_view
        if self.fused_select is None:                         # the library's sequence: one trip through the binding (uq_step)
            self._check_devices(g)
            if self._step_call is None:                      # addresses of my own buffers, marshalled once
                ptr = lambda t: None if t is None else t.data_ptr()
                arr, N = B._scales(self.scales) if self.multi else (None, 0)
                self._step_call = (B.lib().uq_step, self.layout.ref(), arr, N,
                                   (ptr(self.W), ptr(self.idx), ptr(self.lev), ptr(self.out), ptr(self.S),
                                    ptr(self.status), ptr(self.workspace), self.workspace.numel()))
            fn, ref, arr, N, tail = self._step_call
            rc = fn(ref, g.data_ptr(), self.norm, self.s, arr, N, self.idx_bits, seed, self.rng_bits, self.fmt, *tail,
                    B._stream())
            if rc != B.UQ_OK:
                raise B.UqError("uq_step", rc)
            return self._out_view
        # the caller's choice of where selection runs, call by call
        self.agree_scale(g)
        if self.fused_select:                                 # inside the encoder's kernel
            if self.S is None:                                # ... and aggregation + reconstruction too, where it can
                self.select_encode_decode(g, seed)
            else:
                self.select_encode(g, seed)
                self.aggregate_decode()
            return self.out[: self.d]
        if self.multi:
            self.select_scale(g)
        if self.S is None:
            self.encode_decode(g, seed)
        else:
            self.encode(g, seed)
            self.aggregate_decode()
        return self.out[: self.d]

    def _check_devices(self, g: torch.Tensor) -> None:
        """The checks of the marshalling wrappers for the paths that call the library directly: the
        gradients have the layout's shape, and they, this object's buffers and the current device
        (on whose current stream the kernels are launched) are one and the same device."""
        self.layout.check_g(g)
        if not g.is_cuda:
            raise ValueError("uq: tensors must live on a CUDA device")
        current = torch.cuda.current_device()
        B.require_current_device(g.device.index, current, "g")
        B.require_current_device(self.device.index, current, "the quantizer")

    def kernels_per_step(self) -> int:
        """Kernel launches one step enqueues (norm partials + finalize, [select], encode, decode; the
        last two are one kernel when the encoder also aggregates and reconstructs)."""
        if self.one_kernel:
            return 1
        inside = self.selects_inside
        separate_select = self.multi and (not inside or self.M > 8) and self.d > 0
        tail = 0 if self.d == 0 else 1 if self.fused_decode else 2
        return (2 if self.d > 0 else 1) + (1 if separate_select else 0) + tail

    def status_bits(self) -> int:
        """Synchronizes and returns the device status word (0 = clean)."""
        bits = int(self.status.item())
        if bits & B.UQ_STATUS_TIMEOUT and self.small_workspace is not None:   # a barrier wait ran out: its counters are not back at zero
            self.small_workspace.zero_()
        return bits


class RandKQuantizer:
    """GlobalRandKMaxNorm / GlobalRandKMaxNormMultiScale: the K coordinates of this step's shared
    choice are gathered into a compact buffer, the dense quantizer (single- or multi-scale) runs
    on it as one vector, and the K reconstructed values are scattered back."""

    def __init__(self, M: int, d: int, K: int, dtype: torch.dtype = torch.float32, **quantizer_args):
        if not 0 <= K <= d:
            raise ValueError("uq: K must lie in 0..d")
        quantizer_args.pop("seg_off", None)                  # the K-vector is one vector with one scale
        dev = torch.device(quantizer_args.get("device", "cuda"))
        self.M, self.d, self.K = M, d, K
        self.dense_layout = B.Layout(M, d, -(-d // 32) * 32, dtype, None)
        self.inner = Quantizer(M, K, dtype, **quantizer_args)
        self.sel = torch.empty(max(K, 1), dtype=torch.int64, device=dev)
        self.gk = torch.empty((M, self.inner.stride), dtype=dtype, device=dev)
        self.status = self.inner.status

    def gather(self, g: torch.Tensor, seed: int) -> None:
        B.uq_randk_gather(self.dense_layout, g, self.K, seed, self.sel, self.gk, self.status)

    def quantize(self, seed: int) -> torch.Tensor:
        """Agree-scale, [select], encode, aggregate + reconstruct on the compact buffer -> [K] values."""
        return self.inner.step(self.gk, seed)

    def scatter(self, out: torch.Tensor) -> None:
        B.uq_randk_scatter(self.d, self.K, self.sel, self.inner.out, out, self.status)

    def clear(self, out: torch.Tensor) -> None:
        """Zero the entries of ``out`` that the last scatter wrote."""
        B.uq_randk_scatter(self.d, self.K, self.sel, None, out, self.status)

    def update(self, theta: torch.Tensor, lr: float) -> None:
        B.uq_randk_update(self.d, self.K, self.sel, self.inner.out, theta, lr, self.status)

    def step(self, g: torch.Tensor, out: torch.Tensor, seed: int = 0) -> torch.Tensor:
        """g: [M, stride] gradients -> out (dense [d], zero off the chosen set if it was zero before)."""
        self.gather(g, seed)
        self.quantize(seed)
        self.scatter(out)
        return out

    def kernels_per_step(self) -> int:
        return 2 + self.inner.kernels_per_step() if self.K > 0 else 1

    def status_bits(self) -> int:
        return int(self.status.item())


def from_workload(w, keep_sums: bool = False, device="cuda", fused_select: Optional[bool] = None,
                  one_kernel: Optional[bool] = None) -> Quantizer:
    """A Quantizer configured like a ``workloads.Workload``."""
    from . import workloads as wl
    seg = wl.segment_offsets(w)
    return Quantizer(
        M=w.M, d=w.d, dtype=torch.float32 if w.dtype == wl.F32 else torch.bfloat16, seg_off=seg, s=w.s,
        scales=list(w.scales) if w.quantizer == "multi" else None,
        fmt={"i8": B.UQ_FMT_I8, "i4x2": B.UQ_FMT_I4X2, "i2x4": B.UQ_FMT_I2X4, "i6p": B.UQ_FMT_I6P}[w.fmt], idx_bits=w.idx_bits,
        norm=B.UQ_NORM_L2 if w.norm == wl.NORM_L2 else B.UQ_NORM_LINF, rng_bits=w.rng_bits,
        keep_sums=keep_sums, device=device, fused_select=fused_select, one_kernel=one_kernel)


def randk_from_workload(w, K: int, device="cuda") -> RandKQuantizer:
    """A RandKQuantizer with the quantizer settings of a ``workloads.Workload`` (its segments do
    not apply: the K chosen coordinates form one vector)."""
    from . import workloads as wl
    return RandKQuantizer(
        w.M, w.d, K, torch.float32 if w.dtype == wl.F32 else torch.bfloat16, s=w.s,
        scales=list(w.scales) if w.quantizer == "multi" else None,
        fmt={"i8": B.UQ_FMT_I8, "i4x2": B.UQ_FMT_I4X2, "i2x4": B.UQ_FMT_I2X4, "i6p": B.UQ_FMT_I6P}[w.fmt], idx_bits=w.idx_bits,
        norm=B.UQ_NORM_L2 if w.norm == wl.NORM_L2 else B.UQ_NORM_LINF, rng_bits=w.rng_bits, device=device)
