"""uq_agree_scale_static: the shared scale computed with the scratch array built into the
library, for callers that have no way to allocate a workspace.

Collected last on purpose (the file name sorts after every other test file), so a run that stops
at the first failure has already exercised everything else.  The checks depend on nothing the
other tests leave behind: they pass in a fresh process and after the full suite alike.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import from_workload


def _device_gradients(w):
    g = torch.from_numpy(wl.generate(w))
    return (g.view(torch.bfloat16) if w.dtype == wl.BF16 else g).cuda()


@pytest.mark.gpu
def test_static_scratch_matches_the_workspace_entry_point_on_consecutive_calls():
    """Two calls in a row through the C ABI, on different shapes, dtypes and norms, so the second
    one runs on whatever the first left in the shared array.  Both must reproduce
    uq_agree_scale (same kernels, same summation order: the scales agree bit for bit, which is
    inside the 1-ulp bar the parity tests use for the L2 scale)."""
    cases = [wl.scaled("c2", 300_007), wl.scaled("c5", 77_777, norm=wl.NORM_LINF), wl.scaled("c4", 1 << 20)]
    for w in cases + cases[::-1]:
        q = from_workload(w)
        g = _device_gradients(w)
        q.agree_scale(g)                                   # existing entry point, caller's workspace
        want = q.W.clone()
        oracle_W = o.agree_scale(wl.generate(w)[:, : w.d], wl.segment_offsets(w),
                                 o.NORM_LINF if w.norm == wl.NORM_LINF else o.NORM_L2)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for _ in range(2):
            got = torch.full_like(want, -1.0)
            B.uq_agree_scale_static(q.layout, g, q.norm, got, status)
            torch.cuda.synchronize()
            ulp = np.abs(got.cpu().numpy().view(np.int32).astype(np.int64) - want.cpu().numpy().view(np.int32))
            assert ulp.max() <= 1 and ulp.max() == 0
            ulp_oracle = np.abs(got.cpu().numpy().view(np.int32).astype(np.int64) - oracle_W.view(np.int32))
            assert ulp_oracle.max() <= (0 if w.norm == wl.NORM_LINF else 1)      # the parity tests' bar for the scale
        assert int(status.item()) == 0 and float(want.max()) > 0


@pytest.mark.gpu
def test_static_scratch_reports_bad_data_like_the_original():
    w = wl.scaled("c1", 50_000)
    g = _device_gradients(w)
    g[1, 777] = float("nan")
    q = from_workload(w)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.uq_agree_scale_static(q.layout, g, q.norm, q.W, status)
    assert int(status.item()) & B.UQ_STATUS_NONFINITE


def test_layouts_beyond_the_built_in_scratch_are_refused_before_any_launch():
    """M * (ceil(d / 8192) + nseg) * 8 bytes must fit 4 MiB; the check comes first, so this
    runs without a GPU (the pointers are never used)."""
    lib = B.lib()
    p = 0x10000
    big = B.uq_layout(d=1 << 33, worker_stride=1 << 33, seg_off=None, M=8, nseg=1, dtype=B.UQ_F32, worker0=0, coord0=0)
    assert lib.uq_workspace_bytes(C.byref(big)) > B.STATIC_SCRATCH_BYTES
    assert lib.uq_agree_scale_static(C.byref(big), p, B.UQ_NORM_L2, p, None, None) == B.UQ_ERR_WORKSPACE
    bad = B.uq_layout(d=100, worker_stride=100, seg_off=None, M=8, nseg=1, dtype=B.UQ_F32, worker0=0, coord0=0)
    assert lib.uq_agree_scale_static(C.byref(bad), p, B.UQ_NORM_L2, p, None, None) == B.UQ_ERR_BAD_ARG
    assert b"workspace" in lib.uq_error_string(B.UQ_ERR_WORKSPACE)
