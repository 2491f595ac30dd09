"""uq_step_small: the whole step of either quantizer as one cooperative kernel, against the oracle
and against the separate calls."""
import ctypes as C
import dataclasses

import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import Quantizer, from_workload
from parity import _check_parity, run_gpu, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("d", [1, 7, 8, 9, 255, 2049, 100_003, 1 << 20])
@pytest.mark.parametrize("M,dtype,norm,fmt,s,rng_bits", [
    (2, wl.F32, wl.NORM_LINF, "i8", 127, 16), (1, wl.F32, wl.NORM_L2, "i8", 100, 32), (3, wl.BF16, wl.NORM_L2, "i4x2", 7, 16),
    (8, wl.BF16, wl.NORM_LINF, "i2x4", 1, 32), (5, wl.F32, wl.NORM_L2, "i4x2", 5, 32), (8, wl.F32, wl.NORM_L2, "i8", 127, 16),
])
def test_one_kernel_matches_the_oracle(d, M, dtype, norm, fmt, s, rng_bits):
    w = wl.scaled("c1", d, M=M, dtype=dtype, norm=norm, fmt=fmt, s=s, scales=(s,), rng_bits=rng_bits, seed=d + M)
    r = _check_parity(w, wl.generate(w), None, "one")
    assert r["q"].one_kernel and r["q"].kernels_per_step() == 1


@pytest.mark.parametrize("name,d,M", [("c1", 1 << 20, 2), ("c4", 300_007, 8), ("c1", 5_000_011, 2)])
def test_one_kernel_equals_the_separate_calls(name, d, M):
    """Same levels, sums and reconstruction bit for bit; W identical for the maximum norm and within
    one unit in the last place for the Euclidean one (another fixed order of additions).  The last
    case is larger than the resident grid: several units per thread."""
    for norm in (wl.NORM_LINF, wl.NORM_L2):
        w = wl.scaled(name, d, M=M, norm=norm)
        g_np = wl.generate(w)
        one, sep = run_gpu(w, g_np, mode="one"), run_gpu(w, g_np, mode="separate")
        assert one["q"].one_kernel and not sep["q"].one_kernel
        assert one["status"] == 0 and sep["status"] == 0
        if norm == wl.NORM_LINF:
            assert np.array_equal(one["W"], sep["W"])
        else:
            assert abs(int(one["W"].view(np.int32)[0]) - int(sep["W"].view(np.int32)[0])) <= 1
        if np.array_equal(one["W"], sep["W"]):
            nb = w.d >> {"i8": 0, "i4x2": 1}[w.fmt]
            assert np.array_equal(one["lev"][:, :nb], sep["lev"][:, :nb])
            assert np.array_equal(one["S"], sep["S"]) and np.array_equal(one["out"], sep["out"])


def test_the_library_picks_the_one_kernel_step_by_size():
    small = from_workload(wl.scaled("c1", 100_000, M=2))
    big = from_workload(wl.scaled("c1", 2_000_000, M=2))              # 16 MB of gradients
    segmented = from_workload(wl.scaled("c2", 100_000, M=2))
    multi = from_workload(wl.scaled("c3", 100_000, M=4, segments="one"))
    assert small.one_kernel and multi.one_kernel and not big.one_kernel and not segmented.one_kernel
    with pytest.raises(ValueError):
        from_workload(wl.scaled("c2", 100_000, M=2), one_kernel=True)


def test_unsupported_configurations_are_refused():
    g = torch.zeros((9, 128), device="cuda")
    ws = torch.zeros(B.uq_workspace_bytes_small(), dtype=torch.uint8, device="cuda")
    W, out = torch.zeros(1, device="cuda"), torch.zeros(128, device="cuda")
    lev = torch.empty((9, 128), dtype=torch.int8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.UqError) as e:
        B.uq_step_small(B.Layout(9, 100, 128, torch.float32), g, B.UQ_NORM_L2, 127, None, 0, 0, 16, B.UQ_FMT_I8, W, None, lev, out,
                        None, st, ws)
    assert e.value.code == B.UQ_ERR_UNSUPPORTED
    lay = B.Layout(2, 100, 128, torch.float32)
    lev6 = torch.empty((2, lay.level_row_bytes(B.UQ_FMT_I6P)), dtype=torch.int8, device="cuda")
    with pytest.raises(B.UqError) as e:
        B.uq_step_small(lay, g[:2].contiguous(), B.UQ_NORM_L2, 31, None, 0, 0, 16, B.UQ_FMT_I6P, W, None, lev6, out, None, st, ws)
    assert e.value.code == B.UQ_ERR_UNSUPPORTED
    with pytest.raises(B.UqError) as e:
        B.uq_step_small(lay, g[:2].contiguous(), B.UQ_NORM_L2, 127, None, 0, 0, 16, B.UQ_FMT_I8, W, None, lev[:2].contiguous(), out,
                        None, st, ws[:64])
    assert e.value.code == B.UQ_ERR_WORKSPACE
    with pytest.raises(B.UqError) as e:                       # a wait that runs out must be able to say so
        B.uq_step_small(lay, g[:2].contiguous(), B.UQ_NORM_L2, 127, None, 0, 0, 16, B.UQ_FMT_I8, W, None, lev[:2].contiguous(), out,
                        None, None, ws)
    assert e.value.code == B.UQ_ERR_BAD_ARG


def test_draws_are_keyed_by_worker_and_coordinate_of_the_job():
    """layout.worker0 / coord0 as in uq_encode_single: a piece of a larger job."""
    d, M, worker0, coord0 = 70_003, 3, 5, 1 << 20
    w = wl.scaled("c1", d, M=M, norm=wl.NORM_L2)
    g_np = wl.generate(w)
    g = to_device(w, g_np)
    lay = B.Layout(M, d, g.shape[1], torch.float32, None, worker0=worker0, coord0=coord0)
    W, out = torch.zeros(1, device="cuda"), torch.zeros(d, device="cuda")
    lev = torch.zeros((M, g.shape[1]), dtype=torch.int8, device="cuda")
    ws = torch.zeros(B.uq_workspace_bytes_small(), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.uq_step_small(lay, g, B.UQ_NORM_L2, 127, None, 0, 77, 16, B.UQ_FMT_I8, W, None, lev, out, None, status, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = o.encode_single(g_np[:, :d], W.cpu().numpy(), 127, 77, 16, worker0=worker0, coord0=coord0)
    assert np.array_equal(lev.cpu().numpy()[:, :d], want)
    assert np.array_equal(out.cpu().numpy(), o.decode(o.aggregate(want), M, W.cpu().numpy(), s=127))


def test_non_finite_input_sets_the_status_word():
    w = wl.scaled("c1", 10_000, M=2, norm=wl.NORM_L2)
    g_np = wl.generate(w)
    g_np[1, 1234] = np.inf
    q = from_workload(w, one_kernel=True)
    q.step(to_device(w, g_np), 0)
    assert q.status_bits() & B.UQ_STATUS_NONFINITE and not q.status_bits() & B.UQ_STATUS_TIMEOUT


def test_steps_back_to_back():
    """Two hundred one-kernel steps enqueued without a host synchronization (every kernel leaves the
    barrier's counters zero for the next), each with its own seed; the last is checked."""
    w = wl.scaled("c1", 300_001, M=4)
    g_np = wl.generate(w)
    q = from_workload(w, keep_sums=True, one_kernel=True)
    g = to_device(w, g_np)
    for k in range(200):
        q.step(g, k)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    W = q.W.cpu().numpy()
    lev = o.encode_single(g_np[:, : w.d], W, w.s, 199, w.rng_bits)
    assert np.array_equal(q.lev.cpu().numpy()[:, : w.d], lev)
    assert np.array_equal(q.S.cpu().numpy()[: w.d], o.aggregate(lev))


def test_the_wait_at_the_barrier_is_bounded():
    """A wait that cannot be satisfied ends by itself: with the arrival counter started just below
    the wrap of its 32 bits, the CTAs that arrive after the wrap read a count that never reaches the
    grid size.  They give up after their poll limit (about a second), set UQ_STATUS_TIMEOUT and
    return; the context stays usable and, with the scratch zeroed again, the next step is right."""
    w = wl.scaled("c1", 1 << 20, M=2)
    g_np = wl.generate(w)
    q = from_workload(w, keep_sums=True, one_kernel=True)
    g = to_device(w, g_np)
    q.small_workspace[:4] = torch.tensor([0xC0, 0xFF, 0xFF, 0xFF], dtype=torch.uint8)     # 2^32 - 64, little endian
    q.step(g, 0)
    bits = q.status_bits()                       # synchronizes; zeroes the scratch after a timeout
    assert bits & B.UQ_STATUS_TIMEOUT
    assert int(q.small_workspace[:64].sum().item()) == 0
    q.status.zero_()
    _ = q.step(g, w.seed)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    lev = o.encode_single(g_np[:, : w.d], q.W.cpu().numpy(), w.s, w.seed, w.rng_bits)
    assert np.array_equal(q.lev.cpu().numpy()[:, : w.d], lev)


@pytest.mark.parametrize("d", [1, 9, 255, 2049, 100_003, 1 << 20])
@pytest.mark.parametrize("M,dtype,norm,fmt,scales,idx_bits,rng_bits", [
    (2, wl.F32, wl.NORM_L2, "i8", (127, 1016, 8128, 65024), 2, 16), (3, wl.BF16, wl.NORM_L2, "i8", tuple(127 * 8 ** k for k in range(8)), 4, 16),
    (8, wl.F32, wl.NORM_LINF, "i4x2", (7, 112), 1, 32), (5, wl.BF16, wl.NORM_LINF, "i2x4", (1, 16, 256), 8, 32),
    (1, wl.F32, wl.NORM_L2, "i4x2", tuple(5 * 3 ** k for k in range(16)), 4, 32), (4, wl.BF16, wl.NORM_L2, "i8", (100,), 2, 16),
])
def test_one_kernel_multi_scale_matches_the_oracle(d, M, dtype, norm, fmt, scales, idx_bits, rng_bits):
    w = wl.scaled("c3", d, M=M, segments="one", dtype=dtype, norm=norm, fmt=fmt, s=scales[0], scales=scales, idx_bits=idx_bits,
                  rng_bits=rng_bits, seed=3 * d + M)
    r = _check_parity(w, wl.generate(w), None, "one")
    assert r["q"].one_kernel and r["q"].multi and r["q"].kernels_per_step() == 1


@pytest.mark.parametrize("name,d,M", [("c3", 1 << 20, 2), ("c5", 700_001, 8), ("c3", 5_000_011, 2)])
def test_one_kernel_multi_scale_equals_the_separate_calls(name, d, M):
    w = wl.scaled(name, d, M=M, segments="one", norm=wl.NORM_LINF)             # same W bits on both sides
    g_np = wl.generate(w)
    one, sep = run_gpu(w, g_np, mode="one"), run_gpu(w, g_np, mode="separate")
    assert one["q"].one_kernel and not sep["q"].one_kernel and one["status"] == 0 and sep["status"] == 0
    assert np.array_equal(one["W"], sep["W"])
    assert np.array_equal(one["idx"][: w.d * w.idx_bits // 8], sep["idx"][: w.d * w.idx_bits // 8])
    assert np.array_equal(one["lev"][:, : w.d], sep["lev"][:, : w.d])
    assert np.array_equal(one["S"], sep["S"]) and np.array_equal(one["out"], sep["out"])


def test_multi_scale_steps_back_to_back():
    w = wl.scaled("c5", 300_001, M=4, segments="one")
    g_np = wl.generate(w)
    q = from_workload(w, keep_sums=True, one_kernel=True)
    g = to_device(w, g_np)
    for k in range(100):
        q.step(g, k)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    W = q.W.cpu().numpy()
    idx = o.select_scale_multi(g_np[:, : w.d], W, w.scales)
    lev = o.encode_multi(g_np[:, : w.d], W, w.scales, idx, 99, w.rng_bits)
    assert np.array_equal(q.lev.cpu().numpy()[:, : w.d], lev)
    assert np.array_equal(q.S.cpu().numpy()[: w.d], o.aggregate(lev))
    assert np.array_equal(q.out.cpu().numpy()[: w.d], o.decode(o.aggregate(lev), w.M, W, scales=w.scales, idx=idx))


def test_agree_scale_between_steps_does_not_disturb_the_barrier():
    """A one-kernel quantizer whose separate stages are called between its steps (as the benchmark
    does): the norm kernels' scratch and the step's barrier counters are different buffers, so every
    step still waits at its barrier and computes its own W.  Different gradients every step, L2
    norm (a stale or half-written partial would change W), each step compared with the oracle."""
    w = wl.scaled("c1", 300_001, M=5, norm=wl.NORM_L2)
    q = from_workload(w, keep_sums=True, one_kernel=True)
    assert q.one_kernel and q.small_workspace.data_ptr() != q.workspace.data_ptr()
    for step in range(6):
        g_np = wl.generate(dataclasses.replace(w, data_seed=w.data_seed + step)) * np.float32(1 + step)
        g = to_device(w, g_np)
        other = to_device(w, wl.generate(dataclasses.replace(w, data_seed=77 + step)))
        q.agree_scale(other)                                  # the separate call, on other data, right before the step
        q.step(g, 1000 + step)
        torch.cuda.synchronize()
        assert q.status_bits() == 0
        W = q.W.cpu().numpy()
        W_ref = o.agree_scale(g_np[:, : w.d], None, o.NORM_L2)
        assert np.abs(W.view(np.int32).astype(np.int64) - W_ref.view(np.int32)).max() <= 1
        lev = o.encode_single(g_np[:, : w.d], W, w.s, 1000 + step, w.rng_bits)
        assert np.array_equal(q.lev.cpu().numpy()[:, : w.d], lev)
        assert np.array_equal(q.S.cpu().numpy()[: w.d], o.aggregate(lev))
        assert int(q.small_workspace[:64].sum().item()) == 0  # the counters are back at zero after every step
