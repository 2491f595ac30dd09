"""GlobalRandK on the GPU against the oracle: the shared coordinate choice and the gather are
compared bit for bit, the dense stages run on the compact buffer with the usual parity bar, and
the scatter / sparse update are compared element by element."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import randk_from_workload
from parity import FP32_RTOL, check_parity, to_device

pytestmark = pytest.mark.gpu


def _randk(w, K):
    return randk_from_workload(w, K)


@pytest.mark.parametrize("name,d,K,M", [
    ("c2", 2_100_003, 10_000, 8), ("c3", 2_100_003, 10_000, 8), ("c4", 300_007, 4_097, 16),
    ("c5", 1_000_003, 10_000, 8), ("c1", 70_001, 70_001, 2), ("c2", 1000, 1, 3), ("c3", 33, 32, 2),
    ("c2", 5, 3, 1), ("c2", 1, 1, 2), ("c2", 100_000, 0, 2),
])
def test_randk_step_matches_oracle(name, d, K, M):
    w = wl.scaled(name, d, M=M)
    g = wl.generate(w)
    seed = 1234 + d
    rq = _randk(w, K)
    g_dev = to_device(w, g)
    out = torch.full((d,), 7.0, device="cuda")
    rq.step(g_dev, out, seed)
    torch.cuda.synchronize()
    assert rq.status_bits() == 0

    sel = o.randk_indices(d, K, seed)
    assert np.array_equal(rq.sel.cpu().numpy()[:K], sel)
    gk = o.randk_gather(g[:, :d], sel)
    gk_full = gk.base if gk.base is not None else gk
    got_gk = rq.gk.view(torch.int16 if w.dtype == wl.BF16 else torch.float32).cpu().numpy()
    assert np.array_equal(got_gk.view(gk_full.dtype)[:, : gk_full.shape[1]], gk_full[:, : got_gk.shape[1]])
    if K == 0:
        assert (out.cpu().numpy() == 7).all()
        return
    # the dense stages on the compact buffer: the K-vector is one vector with one scale
    wk = dataclasses.replace(w, d=K, segments="one", name=f"{w.name}/randk")
    r = check_parity(wk, np.ascontiguousarray(gk_full), seed)
    assert np.array_equal(rq.inner.out.cpu().numpy()[:K], r["out"])          # the pipeline ran the same thing
    want = np.full(d, 7.0, dtype=np.float32)
    o.randk_scatter(sel, r["ref"]["out"], want)
    got = out.cpu().numpy()
    assert np.allclose(got, want, rtol=FP32_RTOL, atol=0)
    # clearing the chosen entries, then the sparse parameter update
    rq.clear(out)
    want[sel] = 0
    assert np.array_equal(out.cpu().numpy(), want)
    theta0 = np.random.default_rng(d).standard_normal(d).astype(np.float32)
    theta = torch.from_numpy(theta0).cuda()
    rq.update(theta, 0.1)
    assert np.array_equal(theta.cpu().numpy(), o.randk_update(sel, r["out"], theta0, 0.1))


def test_choice_depends_on_the_seed_only():
    """Two dense layouts with different data, worker counts and element types choose the same
    coordinates at the same seed (workers need no communication to agree), another seed differs."""
    d, K = 500_009, 10_000
    sels = []
    for name, M in (("c2", 8), ("c5", 3)):
        w = wl.scaled(name, d, M=M)
        rq = _randk(w, K)
        rq.gather(to_device(w, wl.generate(w)), 77)
        sels.append(rq.sel.cpu().numpy()[:K].copy())
    assert np.array_equal(sels[0], sels[1]) and len(np.unique(sels[0])) == K
    rq.gather(to_device(w, wl.generate(w)), 78)
    assert not np.array_equal(rq.sel.cpu().numpy()[:K], sels[0])


def test_selection_beyond_32_bit_indices():
    """d above 2^32: the permutation runs on 33 bits and the gather addresses with 64-bit offsets.
    The buffer is left uninitialised (13 GB of bf16): only addresses and raw bits are compared."""
    d, K = 3 * 2**31 + 5, 4096
    stride = -(-d // 32) * 32
    g = torch.empty((1, stride), dtype=torch.bfloat16, device="cuda")
    lay = B.Layout(1, d, stride, torch.bfloat16)
    sel = torch.empty(K, dtype=torch.int64, device="cuda")
    gk = torch.empty((1, K), dtype=torch.bfloat16, device="cuda")
    B.uq_randk_gather(lay, g, K, 5, sel, gk)
    want = o.randk_indices(d, K, 5)
    assert np.array_equal(sel.cpu().numpy(), want) and want.max() >= 2**32
    assert torch.equal(gk.view(torch.int16)[0], g.view(torch.int16)[0, torch.from_numpy(want).cuda()])


def test_bad_indices_are_skipped_and_reported():
    d, K = 100, 6
    sel = torch.tensor([3, -1, 99, 100, 2**40, 0], dtype=torch.int64, device="cuda")
    vals = torch.arange(1, K + 1, dtype=torch.float32, device="cuda")
    buf = torch.full((d + 16,), 7.0, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.uq_randk_scatter(d, K, sel, vals, buf[8: 8 + d], status)
    got = buf.cpu().numpy()
    want = np.full(d + 16, 7.0, dtype=np.float32)
    want[8 + 3], want[8 + 99], want[8 + 0] = 1, 3, 6
    assert np.array_equal(got, want) and int(status.item()) == B.UQ_STATUS_BAD_INDEX


def test_randk_argument_checks():
    w = wl.scaled("c2", 1000, M=2)
    rq = _randk(w, 10)
    g = to_device(w, wl.generate(w))
    with pytest.raises(B.UqError):
        B.uq_randk_gather(rq.dense_layout, g, 1001, 0, torch.empty(1001, dtype=torch.int64, device="cuda"),
                          torch.empty((2, 1024), device="cuda"))              # K > d
    with pytest.raises(B.UqError):
        B.uq_randk_gather(rq.dense_layout, g, 10, 0, rq.sel, torch.empty((2, 40), device="cuda"))   # stride % 32
    with pytest.raises(B.UqError):
        B.uq_randk_update(1000, 10, rq.sel, rq.inner.out, torch.zeros(1000, device="cuda"), float("nan"))
