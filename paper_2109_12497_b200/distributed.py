"""Algorithm 1 / 2 with the M workers spread over processes (one process per GPU).

Every process holds ``M_local`` of the job's ``M = world_size * M_local`` gradients.  The paper's
three all-reduces become three exchanges between processes:

  max of the norm        local ``uq_agree_scale``            -> all-reduce(MAX) of W[nseg]
  min of the scale index local ``uq_select_scale_multi``     -> all-gather of the packed rows,
                                                                ``uq_index_min`` (field-wise minimum)
  sum of the levels      local ``uq_encode_*`` (draws keyed  -> all-gather of the level rows,
                         by the worker's number in the job)     fused sum + reconstruction over all
                                                                M rows (``uq_decode``)

so every process ends the step with the same reconstructed average, bit for bit the one a single
process holding all M rows computes.  The level rows travel as they are on the wire (int8, or
packed 4-/2-bit): (world_size - 1) * d * bits / 8 bytes received per process and step.

``pull_levels=True`` replaces the last all-gather by peer loads: the level rows live in symmetric
memory (every process maps the others' rows), and after a stream-ordered barrier between the
processes ``uq_decode_rows`` reads all M rows where they are, its own from HBM and the peers' over
NVLink with ordinary loads, while it sums them: exchange and arithmetic in one kernel, no staging
copy of the gathered rows (2 * (world_size - 1) * d * bits / 8 bytes of HBM traffic less per step).
The barriers are one-element NCCL all-reduces, so a peer that never arrives ends in NCCL's own
timeout handling rather than in a kernel of this library waiting on a flag.  This mode needs
GPUs that can map each other's memory; it has run here on a one-rank group only.

``exchange="slices"`` is the reduce-scatter / all-gather form of the last exchange, the one that keeps
the bytes per process constant as the job grows: the coordinates are cut into ``world_size`` slices of
equal length, an all-to-all hands process r every worker's levels of slice r (still in their wire
format), process r sums and reconstructs its slice (``uq_decode`` on the slice's layout: its own
segment table counted from the slice's start, the matching part of W and of the index), and an
all-gather of the reconstructed slices gives every process the whole average (the packed scale
indices are shared the same way: slices exchanged, ``uq_index_min`` on my slice, slices gathered).
Received per process and step: (world_size - 1) / world_size * (M_local * d * bits / 8 + 4 * d) bytes, against
(world_size - 1) * M_local * d * bits / 8 for the gather of whole rows; fewer from world_size 6 on
for 8-bit levels and one worker per process.  Integer sums do not depend on the order of the rows,
so the result is again bit for bit the single-process one.  Rows are padded to a multiple of
``world_size * 128`` coordinates in this mode (``self.stride``), so that every slice of a level row,
of the packed index and of the output starts on a 16-byte boundary.

The exchanges are ``torch.distributed`` collectives (NCCL on GPUs); every arithmetic step is one
call of the C ABI.  ``kernels`` is the module that provides those calls; it defaults to the CUDA
binding and exists so that the exchange logic can be exercised without GPUs by handing in a
stand-in with the same functions (there is no automatic substitution: without the CUDA library
the default raises).
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch
import torch.distributed as dist


SLICE_ALIGN = 128      # coordinates: 16 bytes of a 1-bit index, 32 of a 2-bit level row, 512 of the output


class DistributedQuantizer:
    def __init__(self, M_local: int, d: int, dtype: torch.dtype = torch.float32,
                 seg_off: Optional[Sequence[int]] = None, s: int = 127,
                 scales: Optional[Sequence[int]] = None, fmt: int = 0, idx_bits: int = 0, norm: int = 2,
                 rng_bits: int = 32, group=None, device: str | torch.device = "cuda", kernels=None,
                 pull_levels: bool = False, exchange: Optional[str] = None):
        exchange = exchange or ("pull" if pull_levels else "gather")
        if exchange not in ("gather", "pull", "slices"):
            raise ValueError("uq: exchange is 'gather', 'pull' or 'slices'")
        pull_levels = exchange == "pull"
        if kernels is None:
            from . import binding as kernels
            kernels.lib()                               # fail now if the CUDA library is not built
        self.k = kernels
        self.group = group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.M_local, self.M, self.d, self.dtype = M_local, M_local * self.world, d, dtype
        if self.M > 64:
            raise ValueError("uq: at most 64 workers in a job")
        dev = torch.device(device)
        self.exchange = exchange
        self.stride = -(-d // 32) * 32
        if exchange == "slices":
            if fmt not in (0, 1, 2):
                raise ValueError("uq: the slice exchange needs a level format whose rows are one plane")
            self.slice_coords = max(1, -(-d // (self.world * SLICE_ALIGN))) * SLICE_ALIGN
            self.stride = self.world * self.slice_coords
        self.multi = scales is not None and idx_bits != 0
        self.s = int(scales[0]) if self.multi else int(s)
        self.scales = [int(x) for x in scales] if self.multi else None
        self.fmt, self.idx_bits, self.norm, self.rng_bits = fmt, idx_bits if self.multi else 0, norm, rng_bits
        seg_dev = None
        if seg_off is not None and len(seg_off) > 2:
            seg_dev = torch.as_tensor(np.asarray(seg_off, dtype=np.int64), device=dev)
        # my rows are workers rank*M_local .. of the job; the gathered rows are all of them
        self.local = self.k.Layout(M_local, d, self.stride, dtype, seg_dev, worker0=self.rank * M_local)
        self.total = self.k.Layout(self.M, d, self.stride, dtype, seg_dev)
        nseg = self.local.nseg
        row_bytes = self.local.level_row_bytes(fmt)
        self.W = torch.zeros(nseg, dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.workspace = torch.empty(max(8, self.local.workspace_bytes()), dtype=torch.uint8, device=dev)
        self.pull_levels = pull_levels
        if pull_levels:
            import torch.distributed._symmetric_memory as symm_mem
            self.lev_local = symm_mem.empty((M_local, row_bytes), dtype=torch.int8, device=dev)
            self._mapping = symm_mem.rendezvous(self.lev_local, dist.group.WORLD if group is None else group)
            base = self._mapping.buffer_ptrs                       # where rank r's rows are mapped here
            self.peer_rows = [base[r] + m * row_bytes for r in range(self.world) for m in range(M_local)]
            self._flag = torch.zeros(1, dtype=torch.int32, device=dev)
            self.lev_all = None
        else:
            self.lev_local = torch.empty((M_local, row_bytes), dtype=torch.int8, device=dev)
            self.lev_all = torch.empty((self.M, row_bytes), dtype=torch.int8, device=dev)
        self.idx = self.idx_local = self.idx_rows = None
        if self.multi:
            nb = max(16, self.local.index_bytes(self.idx_bits))
            self.idx_local = torch.empty(nb, dtype=torch.uint8, device=dev)
            self.idx_rows = torch.empty((self.world, nb), dtype=torch.uint8, device=dev)
            self.idx = torch.empty(nb, dtype=torch.uint8, device=dev)
        self.out = torch.empty(max(d, 1), dtype=torch.float32, device=dev)
        if exchange == "slices":
            self._init_slices(seg_off, dev)

    def _init_slices(self, seg_off, dev) -> None:
        """Layout and buffers of my slice: coordinates [c, c + d_r) of every worker's row."""
        P, c = self.slice_coords, self.rank * self.slice_coords
        self.slice_d = d_r = min(max(self.d - c, 0), P)
        seg = np.asarray([0, self.d] if seg_off is None or len(seg_off) <= 2 else seg_off, dtype=np.int64)
        j0 = int(np.searchsorted(seg, c, side="right") - 1) if d_r else 0
        j1 = int(np.searchsorted(seg, c + d_r, side="left")) if d_r else 1      # segments j0 .. j1-1 meet my slice
        sub = np.clip(seg[j0: j1 + 1] - c, 0, d_r)
        sub_dev = torch.as_tensor(sub, device=dev) if len(sub) > 2 else None
        self.slice_layout = self.k.Layout(self.M, d_r, P, self.dtype, sub_dev)
        self.slice_seg = (j0, j1)
        self.slice_bytes = self.slice_layout.level_row_bytes(self.fmt)
        assert self.slice_bytes * self.world == self.local.level_row_bytes(self.fmt)
        self.lev_recv = torch.empty((self.M_local, self.world, self.slice_bytes), dtype=torch.int8, device=dev)
        self.out_slice = torch.zeros(P, dtype=torch.float32, device=dev)
        self.out = self.out_all = torch.empty(self.world * P, dtype=torch.float32, device=dev)
        if self.multi:
            self.idx_slice = torch.empty(P * self.idx_bits // 8, dtype=torch.uint8, device=dev)
        self.lev_all = None

    # the three exchanges ------------------------------------------------------------------------
    def agree_scale(self, g: torch.Tensor) -> None:
        """Algorithm 1 / 2 line "MaxAllReduce Norm"."""
        self.k.uq_agree_scale(self.local, g, self.norm, self.W, self.status, self.workspace)
        dist.all_reduce(self.W, op=dist.ReduceOp.MAX, group=self.group)

    def share_scale_index(self, g: torch.Tensor) -> None:
        """Algorithm 2 lines "Compute coordinate scales" and "Scale sharing"."""
        self.k.uq_select_scale_multi(self.local, g, self.W, self.scales, self.idx_bits, self.idx_local, self.status)
        if self.exchange == "slices":          # the same in reduce-scatter / all-gather form: my slice from everyone,
            nb = self.slice_coords * self.idx_bits // 8                                  # its minimum to everyone
            dist.all_to_all_single(self.idx_rows.view(-1)[: self.world * nb], self.idx_local[: self.world * nb],
                                   group=self.group)
            rows = self.idx_rows.view(-1)[: self.world * nb].view(self.world, nb)
            self.k.uq_index_min(rows, self.idx_bits, self.idx_slice)
            dist.all_gather_into_tensor(self.idx[: self.world * nb], self.idx_slice, group=self.group)
            return
        dist.all_gather_into_tensor(self.idx_rows.view(-1), self.idx_local, group=self.group)
        self.k.uq_index_min(self.idx_rows, self.idx_bits, self.idx)

    def encode(self, g: torch.Tensor, seed: int) -> None:
        if self.multi:
            self.k.uq_encode_multi(self.local, g, self.W, self.scales, self.idx, self.idx_bits, seed, self.rng_bits,
                                   self.fmt, self.lev_local, self.status)
        else:
            self.k.uq_encode_single(self.local, g, self.W, self.s, seed, self.rng_bits, self.fmt, self.lev_local,
                                    self.status)

    def exchange_and_reconstruct(self) -> None:
        """Algorithm 1 / 2 lines "AllReduce gradients" and "Reconstruct gradient": the level rows of
        all processes are gathered as they are on the wire, summed and reconstructed in one kernel."""
        if self.exchange == "slices":
            return self._exchange_slices()
        if self.pull_levels:
            dist.all_reduce(self._flag, group=self.group)          # every process has finished its encoder
            self.k.uq_decode_rows(self.total, self.peer_rows, self.fmt, self.W, self.s, self.scales, self.idx,
                                  self.idx_bits, self.out, None)
            dist.all_reduce(self._flag, group=self.group)          # every process has read my rows
            return
        dist.all_gather_into_tensor(self.lev_all.view(-1), self.lev_local.view(-1), group=self.group)
        self.k.uq_decode(self.total, self.lev_all, self.k.UQ_SRC_LEVELS, self.fmt, self.W, self.s, self.scales,
                         self.idx, self.idx_bits, self.out, None)

    def _exchange_slices(self) -> None:
        """Slice r of every level row goes to process r (one all-to-all per local worker: a row is
        already laid out slice after slice), process r reconstructs slice r from all M rows, and the
        slices are gathered.  The received rows are in (local worker, sender) order, which the
        integer sum does not see."""
        for m in range(self.M_local):
            dist.all_to_all_single(self.lev_recv[m].view(-1), self.lev_local[m], group=self.group)
        if self.slice_d > 0:
            j0, j1 = self.slice_seg
            c = self.rank * self.slice_coords
            idx = None if self.idx is None else self.idx[c * self.idx_bits // 8:]
            self.k.uq_decode(self.slice_layout, self.lev_recv.view(self.M, self.slice_bytes), self.k.UQ_SRC_LEVELS,
                             self.fmt, self.W[j0:j1], self.s, self.scales, idx, self.idx_bits, self.out_slice, None)
        dist.all_gather_into_tensor(self.out_all, self.out_slice, group=self.group)

    def step(self, g: torch.Tensor, seed: int = 0) -> torch.Tensor:
        """g: [M_local, stride] gradients of my workers -> the average gradient of the job [d]."""
        self.agree_scale(g)
        if self.multi:
            self.share_scale_index(g)
        self.encode(g, seed)
        self.exchange_and_reconstruct()
        return self.out[: self.d]

    def wire_bytes_per_step(self) -> int:
        """Bytes this process receives from the others in one step."""
        others = self.world - 1
        if self.exchange == "slices":
            n = others * (self.M_local * self.slice_bytes + 4 * self.slice_coords) + (self.W.numel() * 4 if others else 0)
        else:
            n = others * self.lev_local.numel() + (self.W.numel() * 4 if others else 0)
        if self.multi and self.exchange == "slices":
            n += 2 * others * self.idx_slice.numel()
        elif self.multi:
            n += others * self.idx_local.numel()
        return n
