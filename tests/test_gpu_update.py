"""Parity of the fused aggregate + reconstruct + parameter-update kernel (through the C ABI) with the
oracle: levels -> sums -> g_hat -> SGD step on theta and the momentum buffer."""
import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from parity import FP32_RTOL, check_parity, run_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,d", [("c2", 100_003), ("c3", 70_001), ("c4", 65_537), ("c5", 50_021), ("c1", 5)])
@pytest.mark.parametrize("lr,mu,wd,use_mom", [(0.1, 0.0, 0.0, False), (0.1, 0.9, 5e-4, True), (0.05, 0.9, 0.0, True),
                                              (0.1, 0.0, 5e-4, False)])
def test_fused_update_matches_oracle(name, d, lr, mu, wd, use_mom):
    _fused_update_case(wl.scaled(name, d), lr, mu, wd, use_mom)


def test_fused_update_two_bit_levels():
    _fused_update_case(wl.scaled("c2", 100_003, fmt="i2x4", s=1, scales=(1,)), 0.1, 0.9, 5e-4, True)
    _fused_update_case(wl.scaled("c3", 70_001, fmt="i2x4", s=1, scales=(1, 16, 256)), 0.1, 0.0, 0.0, False)


def _fused_update_case(w, lr, mu, wd, use_mom):
    d = w.d
    r = check_parity(w, wl.generate(w))            # levels, sums and g_hat of the step, compared with the oracle
    q = r["q"]
    rng = np.random.default_rng(d)
    theta0 = rng.standard_normal(w.d).astype(np.float32)
    mom0 = (rng.standard_normal(w.d) * 1e-2).astype(np.float32) if use_mom else None
    pad = 8                                             # 32-byte aligned slices with canaries around them
    theta = torch.full((w.d + 2 * pad,), 7.0, device="cuda"); theta[pad: pad + w.d] = torch.from_numpy(theta0).cuda()
    mom = None
    if use_mom:
        mom = torch.full((w.d + 2 * pad,), 7.0, device="cuda"); mom[pad: pad + w.d] = torch.from_numpy(mom0).cuda()
    ghat = torch.empty(w.d, device="cuda")
    for step in range(2):                               # two steps: the buffers carry state
        B.uq_decode_update(q.layout, q.lev, q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits,
                           theta[pad: pad + w.d], None if mom is None else mom[pad: pad + w.d], lr, mu, wd, ghat)
        torch.cuda.synchronize()
        assert np.array_equal(ghat.cpu().numpy(), r["out"])          # same g_hat as the plain decode ...
        assert np.allclose(ghat.cpu().numpy(), r["ref"]["out"], rtol=FP32_RTOL, atol=0)    # ... and as the oracle's
        theta0, mom0 = o.sgd_update(r["ref"]["out"], theta0, mom0, lr=lr, mu=mu, wd=wd)   # the oracle's g_hat, not the GPU's
        got = theta.cpu().numpy()
        assert np.allclose(got[pad: pad + w.d], theta0, rtol=FP32_RTOL, atol=0)
        assert np.array_equal(got[pad: pad + w.d], theta0)           # same operation order: bit-equal
        assert (got[:pad] == 7).all() and (got[pad + w.d:] == 7).all()
        if use_mom:
            gm = mom.cpu().numpy()
            assert np.array_equal(gm[pad: pad + w.d], mom0) and (gm[:pad] == 7).all() and (gm[pad + w.d:] == 7).all()


def test_update_rejects_bad_arguments():
    w = wl.scaled("c1", 1000)
    q = run_gpu(w, wl.generate(w))["q"]
    theta = torch.zeros(w.d + 8, device="cuda")
    with pytest.raises(B.UqError):
        B.uq_decode_update(q.layout, q.lev, q.fmt, q.W, q.s, None, None, 0, theta[1: 1 + w.d], None, 0.1)   # misaligned
    with pytest.raises(B.UqError):
        B.uq_decode_update(q.layout, q.lev, q.fmt, q.W, q.s, None, None, 0, theta[: w.d], None, float("nan"))
