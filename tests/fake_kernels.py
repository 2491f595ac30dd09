"""A stand-in for ``paper_2109_12497_b200.binding`` that runs on CPU tensors: every call of the
C ABI that the distributed step makes is answered by the CPU oracle.  Test infrastructure only:
it lets the exchange logic (who sends what to whom, which worker numbers key the draws, which M
divides the sum) run under gloo on machines without a GPU.  The arithmetic it produces is the
oracle's, so comparing with the oracle checks the protocol, not the kernels."""
from __future__ import annotations

import numpy as np
import torch

from oracle import uq_oracle as o

UQ_F32, UQ_BF16 = 0, 1
UQ_NORM_LINF, UQ_NORM_L2 = 0, 2
UQ_FMT_I8, UQ_FMT_I4X2, UQ_FMT_I2X4 = 0, 1, 2
UQ_SRC_LEVELS, UQ_SRC_SUMS = 0, 1


def lib():
    return None


class Layout:
    def __init__(self, M, d, worker_stride, dtype, seg_off=None, worker0=0, coord0=0):
        assert coord0 == 0
        self.M, self.d, self.worker_stride, self.dtype, self.seg_off, self.worker0 = M, d, worker_stride, dtype, seg_off, worker0
        self.nseg = 1 if seg_off is None else seg_off.numel() - 1

    def workspace_bytes(self):
        return 8

    def index_bytes(self, idx_bits):
        return self.worker_stride * idx_bits // 8

    def level_row_bytes(self, fmt):
        return self.worker_stride >> fmt

    def seg(self):
        return None if self.seg_off is None else self.seg_off.numpy()


def _g(layout, g):
    a = g.view(torch.int16).numpy().view(np.uint16) if g.dtype == torch.bfloat16 else g.numpy()
    return a[:, : layout.d]


def _unpack_fields(packed: np.ndarray, bits: int, n: int) -> np.ndarray:
    """The first n unsigned fields of `bits` bits, lowest bits first."""
    per = 8 // bits
    shifts = (np.arange(per) * bits).astype(np.uint8)
    return ((packed[..., None] >> shifts) & ((1 << bits) - 1)).reshape(*packed.shape[:-1], -1)[..., :n]


def uq_agree_scale(layout, g, norm, W, status, workspace):
    W.copy_(torch.from_numpy(o.agree_scale(_g(layout, g), layout.seg(), norm)))


def uq_select_scale_multi(layout, g, W, scales, idx_bits, idx, status):
    k = o.select_scale_multi(_g(layout, g), W.numpy(), scales, seg_off=layout.seg())
    packed = o.pack_index(k, idx_bits)
    idx.zero_()
    idx[: packed.size] = torch.from_numpy(packed)


def uq_index_min(rows, idx_bits, idx, nbytes=None):
    n = rows.shape[1] * 8 // idx_bits
    k = o.index_min(_unpack_fields(rows.numpy(), idx_bits, n))
    packed = o.pack_index(k, idx_bits)
    idx[: packed.size] = torch.from_numpy(packed)


def _store_levels(layout, fmt, lev, out):
    packed = {UQ_FMT_I8: lambda x: np.ascontiguousarray(x).view(np.uint8), UQ_FMT_I4X2: o.pack_levels_i4,
              UQ_FMT_I2X4: o.pack_levels_i2}[fmt](lev)
    out.zero_()
    out.view(torch.uint8)[:, : packed.shape[1]] = torch.from_numpy(np.ascontiguousarray(packed))


def uq_encode_single(layout, g, W, s, seed, rng_bits, fmt, lev, status):
    z = o.encode_single(_g(layout, g), W.numpy(), s, seed, rng_bits, seg_off=layout.seg(), worker0=layout.worker0)
    _store_levels(layout, fmt, z, lev)


def uq_encode_multi(layout, g, W, scales, idx, idx_bits, seed, rng_bits, fmt, lev, status):
    k = _unpack_fields(idx.numpy(), idx_bits, layout.d)
    z = o.encode_multi(_g(layout, g), W.numpy(), scales, k, seed, rng_bits, seg_off=layout.seg(), worker0=layout.worker0)
    _store_levels(layout, fmt, z, lev)


def uq_decode(layout, src, src_kind, fmt, W, s, scales, idx, idx_bits, out, S_opt=None):
    assert src_kind == UQ_SRC_LEVELS
    raw = src.view(torch.uint8).numpy()
    if fmt == UQ_FMT_I8:
        lev = raw.view(np.int8)[:, : layout.d]
    else:
        bits = 4 if fmt == UQ_FMT_I4X2 else 2
        u = _unpack_fields(raw, bits, layout.d).astype(np.int16)
        lev = ((u ^ (1 << (bits - 1))) - (1 << (bits - 1))).astype(np.int8)       # sign extension
    S = o.aggregate(np.ascontiguousarray(lev))
    if scales is None:
        r = o.decode(S, layout.M, W.numpy(), s=s, seg_off=layout.seg())
    else:
        r = o.decode(S, layout.M, W.numpy(), scales=scales, idx=_unpack_fields(idx.numpy(), idx_bits, layout.d),
                     seg_off=layout.seg())
    out[: layout.d] = torch.from_numpy(r)
