"""Runs one workload through the CUDA library (C ABI) and through the CPU oracle and compares
them element by element.  Test helper; the two sides share only the input array."""
from __future__ import annotations

import numpy as np
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import from_workload

FP32_RTOL = 1e-6          # the stated bar for the reconstructed fp32 values


def to_device(w, g_np):
    t = torch.from_numpy(g_np)
    if w.dtype == wl.BF16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def run_gpu(w, g_np, seed=None, mode="default"):
    """All stage outputs of the CUDA path as numpy arrays.  mode picks the form of the path:
    "default" (what the library picks: the one-kernel step for small gradients, else uq_step),
    "fused" (multi-scale: selection and encoding as one call, uq_select_encode_multi), "one" (the
    whole step as one cooperative kernel), "separate" (never the one-kernel step), "nosums" (the step
    without the integer sums among its outputs: quantization, aggregation and reconstruction as one
    call, uq_encode_decode; the sums compared below then come from uq_aggregate over its levels),
    "fused_nosums" (multi-scale: everything behind the scale agreement as one call,
    uq_select_encode_decode_multi), "auto_nosums" (uq_step without the integer sums: the form a user
    gets, in which the library picks the fewest kernels itself)."""
    one_kernel = {"one": True, "separate": False, "fused": False, "nosums": False, "fused_nosums": False,
                  "auto_nosums": False}.get(mode)               # else: the library decides by size
    nosums = mode in ("nosums", "fused_nosums", "auto_nosums")
    # where selection runs: the library's choice (uq_step), or the caller's, call by call
    fused_select = None if mode in ("default", "auto_nosums") else mode in ("fused", "fused_nosums")
    q = from_workload(w, keep_sums=not nosums, fused_select=fused_select, one_kernel=one_kernel)
    g = to_device(w, g_np)
    q.step(g, w.seed if seed is None else seed)
    if nosums:
        q.S = torch.empty(max(w.d, 1), dtype=torch.int32, device="cuda")
        B.uq_aggregate(q.layout, q.lev, q.fmt, q.S)
    torch.cuda.synchronize()
    res = dict(
        W=q.W.cpu().numpy(), lev=q.lev.cpu().numpy().view(np.uint8), S=q.S.cpu().numpy()[: w.d],
        out=q.out.cpu().numpy()[: w.d], status=q.status_bits(), q=q,
    )
    if q.multi:
        res["idx"] = q.idx.cpu().numpy()
    return res


def run_oracle(w, g_np, W=None, seed=None):
    """The oracle's outputs in the library's wire formats.  W given: skip the norm (chain rule:
    downstream parity is conditioned on the scale bits)."""
    seed = w.seed if seed is None else seed
    g = g_np[:, : w.d]
    seg = wl.segment_offsets(w)
    norm = o.NORM_L2 if w.norm == wl.NORM_L2 else o.NORM_LINF
    W_own = o.agree_scale(g, seg, norm)
    W = W_own if W is None else W
    res = dict(W=W_own)
    if w.quantizer == "multi":
        idx = o.select_scale_multi(g, W, w.scales, seg_off=seg)
        lev = o.encode_multi(g, W, w.scales, idx, seed, w.rng_bits, seg_off=seg)
        S = o.aggregate(lev)
        out = o.decode(S, w.M, W, scales=w.scales, idx=idx, seg_off=seg)
        res["idx"] = o.pack_index(idx, w.idx_bits)
        res["idx_raw"] = idx
    else:
        lev = o.encode_single(g, W, w.s, seed, w.rng_bits, seg_off=seg)
        S = o.aggregate(lev)
        out = o.decode(S, w.M, W, s=w.s, seg_off=seg)
    res["lev_raw"] = lev
    if w.fmt == "i4x2":
        res["lev"] = o.pack_levels_i4(lev)
    elif w.fmt == "i2x4":
        res["lev"] = o.pack_levels_i2(lev)
    elif w.fmt == "i6p":
        res["lev"] = o.pack_levels_i6p(lev, -(-w.d // 32) * 32)
    else:
        res["lev"] = np.ascontiguousarray(lev).view(np.uint8)
    res.update(S=S, out=out)
    return res


def ulp_distance(a, b):
    ia = a.view(np.int32).astype(np.int64)
    ib = b.view(np.int32).astype(np.int64)
    return np.abs(ia - ib)


def check_parity(w, g_np, seed=None):
    """Full comparison; returns the GPU result for further checks.  A multi-scale workload runs in
    both forms of its path (see run_gpu), a workload that the one-kernel step takes in both of
    its forms, and every workload also without the integer sums among the outputs (the form in which
    the encoder aggregates and reconstructs itself where it can): each must match the oracle."""
    if w.quantizer == "multi":
        _check_parity(w, g_np, seed, "fused")
        _check_parity(w, g_np, seed, "fused_nosums")
    _check_parity(w, g_np, seed, "nosums")
    _check_parity(w, g_np, seed, "auto_nosums")
    if one_kernel_takes(w):
        _check_parity(w, g_np, seed, "one")
        _check_parity(w, g_np, seed, "separate")
    return _check_parity(w, g_np, seed, "default")


def one_kernel_takes(w) -> bool:
    return len(wl.segment_offsets(w)) == 2 and w.M <= B.SMALL_STEP_MAX_WORKERS and w.fmt in ("i8", "i4x2", "i2x4")


def _check_parity(w, g_np, seed, mode):
    gpu = run_gpu(w, g_np, seed, mode)
    assert gpu["status"] == 0
    ref_own = run_oracle(w, g_np, None, seed)
    # scale: exact for L-infinity; for L2 the binary64 sums may differ in the last bits, which
    # can move the rounded binary32 by one ulp at most
    dist = ulp_distance(gpu["W"], ref_own["W"])
    if w.norm == wl.NORM_LINF:
        assert dist.max(initial=0) == 0
    else:
        assert dist.max(initial=0) <= 1, f"W differs by {dist.max()} ulp"
    # downstream stages are compared with the oracle fed the GPU's scale bits
    ref = ref_own if dist.max(initial=0) == 0 else run_oracle(w, g_np, gpu["W"], seed)
    if w.fmt == "i6p":                       # two planes per row; the rest of a row is padding
        half = (-(-w.d // 32) * 32) // 2
        for a, n in ((0, -(-w.d // 2)), (half, -(-w.d // 4))):
            assert np.array_equal(gpu["lev"][:, a: a + n], ref["lev"][:, a: a + n]), "levels differ"
    else:
        nb_lev = ref["lev"].shape[1]
        assert np.array_equal(gpu["lev"][:, :nb_lev], ref["lev"]), "levels differ"
    if w.quantizer == "multi":
        nb = ref["idx"].size
        assert np.array_equal(gpu["idx"][:nb], ref["idx"]), "scale indices differ"
    assert np.array_equal(gpu["S"], ref["S"]), "integer sums differ"
    assert np.allclose(gpu["out"], ref["out"], rtol=FP32_RTOL, atol=0), "reconstruction differs"
    gpu["ref"] = ref
    gpu["w_ulp"] = int(dist.max(initial=0))
    return gpu
