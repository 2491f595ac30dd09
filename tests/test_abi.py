"""The C-ABI library loads without a GPU, exports everything include/uq.h declares, and its
host-side argument validation rejects bad calls before any launch."""
import ctypes as C
import re
from pathlib import Path

import pytest

from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import build as uq_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    uq_build.build()
    return B.lib()


def declared_functions():
    text = (ROOT / "include" / "uq.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(uq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_constants_match_the_header():
    text = (ROOT / "include" / "uq.h").read_text()
    for name in ("UQ_OK", "UQ_ERR_BAD_ARG", "UQ_ERR_CUDA", "UQ_ERR_UNSUPPORTED", "UQ_ERR_WORKSPACE",
                 "UQ_F32", "UQ_BF16", "UQ_NORM_LINF", "UQ_NORM_L2", "UQ_FMT_I8", "UQ_FMT_I4X2", "UQ_FMT_I2X4", "UQ_FMT_I6P",
                 "UQ_SRC_LEVELS", "UQ_SRC_SUMS", "UQ_STATUS_NONFINITE", "UQ_STATUS_BAD_SEGMENTS",
                 "UQ_STATUS_SCALE_OVERFLOW", "UQ_STATUS_BAD_INDEX", "UQ_STATUS_TIMEOUT"):
        m = re.search(rf"\b{name}\s*=\s*(\d+)", text)
        assert m and int(m.group(1)) == getattr(B, name), name


def _layout(**kw):
    base = dict(d=1000, worker_stride=1024, seg_off=None, M=2, nseg=1, dtype=B.UQ_F32, worker0=0, coord0=0)
    base.update(kw)
    return B.uq_layout(**base)


def test_sizes(lib):
    L = _layout()
    assert lib.uq_workspace_bytes(C.byref(L)) == 2 * (1 + 1) * 8
    assert lib.uq_index_bytes(C.byref(L), 2) == 256 and lib.uq_index_bytes(C.byref(L), 4) == 512
    assert lib.uq_index_bytes(C.byref(L), 3) == 0
    assert lib.uq_workspace_bytes(C.byref(_layout(worker_stride=1000))) == 0      # not a multiple of 32
    assert lib.uq_version() >= 100
    assert lib.uq_error_string(B.UQ_ERR_BAD_ARG) == b"bad argument"


def test_bad_arguments_are_rejected_on_the_host(lib):
    """None of these reaches a launch, so they run without a GPU (pointers are fake but aligned)."""
    p = 0x10000
    ok = _layout()
    bad_layouts = [_layout(M=0), _layout(M=65), _layout(d=-1), _layout(worker_stride=992), _layout(nseg=2),
                   _layout(dtype=5), _layout(worker0=-1), _layout(nseg=0), _layout(coord0=4), _layout(coord0=-8)]
    for L in bad_layouts:
        assert lib.uq_agree_scale(C.byref(L), p, B.UQ_NORM_L2, p, None, p, 1 << 20, None) == B.UQ_ERR_BAD_ARG
        assert lib.uq_encode_single(C.byref(L), p, p, 127, 0, 32, B.UQ_FMT_I8, p, None, None) == B.UQ_ERR_BAD_ARG
    r = C.byref(ok)
    assert lib.uq_agree_scale(r, p, 1, p, None, p, 1 << 20, None) == B.UQ_ERR_BAD_ARG            # norm
    assert lib.uq_agree_scale(r, p, B.UQ_NORM_L2, p, None, p, 8, None) == B.UQ_ERR_WORKSPACE      # too small
    assert lib.uq_agree_scale(r, p, B.UQ_NORM_L2, p, None, None, 1 << 20, None) == B.UQ_ERR_WORKSPACE
    assert lib.uq_agree_scale(r, p + 4, B.UQ_NORM_L2, p, None, p, 1 << 20, None) == B.UQ_ERR_BAD_ARG  # alignment
    for s, fmt in ((0, B.UQ_FMT_I8), (128, B.UQ_FMT_I8), (8, B.UQ_FMT_I4X2), (2, B.UQ_FMT_I2X4), (32, B.UQ_FMT_I6P), (5, 4)):
        assert lib.uq_encode_single(r, p, p, s, 0, 32, fmt, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_encode_single(r, p, p, 127, 0, 24, B.UQ_FMT_I8, p, None, None) == B.UQ_ERR_BAD_ARG  # rng_bits
    assert lib.uq_encode_single(r, p, None, 127, 0, 32, B.UQ_FMT_I8, p, None, None) == B.UQ_ERR_BAD_ARG

    def scales(*v):
        return (C.c_int32 * len(v))(*v)
    for sc, n, bits in ((scales(127, 127), 2, 2), (scales(127, 64), 2, 2), (scales(0, 5), 2, 2),
                        (scales(1, 2, 3, 4, 5), 5, 2), (scales(127, 1016), 2, 3), (scales(127), 0, 2)):
        assert lib.uq_select_scale_multi(r, p, p, sc, n, bits, p, None, None) == B.UQ_ERR_BAD_ARG
        assert lib.uq_encode_multi(r, p, p, sc, n, p, bits, 0, 32, B.UQ_FMT_I8, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_encode_multi(r, p, p, scales(200, 400), 2, p, 2, 0, 32, B.UQ_FMT_I8, p, None, None) \
        == B.UQ_ERR_BAD_ARG                                                                        # s_hat > 127
    assert lib.uq_aggregate(r, p, 7, p, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode(r, p, 2, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode(r, p, B.UQ_SRC_LEVELS, B.UQ_FMT_I8, p, 0, None, 0, None, 0, p, None, None) \
        == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode(r, p, B.UQ_SRC_LEVELS, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p + 4, None, None) \
        == B.UQ_ERR_BAD_ARG


def test_later_entry_points_reject_bad_arguments_on_the_host(lib):
    """The entry points added after the six of the hot path: same rule, nothing is launched."""
    p = 0x10000
    F = C.c_float
    ok, bad = C.byref(_layout()), C.byref(_layout(M=0))
    sc = (C.c_int32 * 2)(127, 1016)
    rows = (C.c_void_p * 2)(p, p)
    assert lib.uq_step(bad, p, B.UQ_NORM_L2, 127, None, 0, 0, 0, 16, B.UQ_FMT_I8, p, None, p, p, None, None, p, 1 << 20,
                       None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_step(ok, p, B.UQ_NORM_L2, 127, None, 0, 0, 0, 16, B.UQ_FMT_I8, p, None, p, p, None, None, p, 8,
                       None) == B.UQ_ERR_WORKSPACE
    small_bytes = lib.uq_workspace_bytes_small()
    assert small_bytes >= 64 + 148 * 8 * 8 * 8
    def small(L, s=127, scales=None, N=0, bits=0, fmt=B.UQ_FMT_I8, out=p, idx=None, ws=small_bytes, status=p):
        return lib.uq_step_small(L, p, B.UQ_NORM_L2, s, scales, N, bits, 0, 16, fmt, p, idx, p, out, None, status, p, ws, None)
    assert small(bad) == B.UQ_ERR_BAD_ARG
    assert small(ok, status=None) == B.UQ_ERR_BAD_ARG                                      # a timeout must be reportable
    assert small(ok, s=128) == B.UQ_ERR_BAD_ARG
    assert small(ok, out=p + 16) == B.UQ_ERR_BAD_ARG                                      # out: 32-byte aligned
    assert small(ok, scales=sc, N=2, bits=3, idx=p) == B.UQ_ERR_BAD_ARG                     # idx_bits
    assert small(ok, scales=sc, N=2, bits=2, idx=None) == B.UQ_ERR_BAD_ARG                  # multi-scale needs idx
    assert small(C.byref(_layout(M=9))) == B.UQ_ERR_UNSUPPORTED
    assert small(ok, s=31, fmt=B.UQ_FMT_I6P) == B.UQ_ERR_UNSUPPORTED
    assert small(ok, ws=64) == B.UQ_ERR_WORKSPACE
    assert small(ok, scales=sc, N=2, bits=2, idx=p, ws=64) == B.UQ_ERR_WORKSPACE
    assert lib.uq_select_encode_multi(ok, p, p, sc, 2, 3, 0, 16, B.UQ_FMT_I8, p, p, None, None) == B.UQ_ERR_BAD_ARG   # idx_bits
    assert lib.uq_select_encode_multi(ok, p, p, sc, 2, 2, 0, 16, B.UQ_FMT_I4X2, p, p, None, None) == B.UQ_ERR_BAD_ARG  # s_hat > 7
    assert lib.uq_select_encode_multi(ok, p, p, sc, 2, 2, 0, 16, B.UQ_FMT_I8, None, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_select_encode_decode_multi(ok, p, p, sc, 2, 3, 0, 16, B.UQ_FMT_I8, p, p, p, None, None) == B.UQ_ERR_BAD_ARG   # idx_bits
    assert lib.uq_select_encode_decode_multi(ok, p, p, sc, 2, 2, 0, 16, B.UQ_FMT_I8, p, p, None, None, None) == B.UQ_ERR_BAD_ARG  # out
    assert lib.uq_select_encode_decode_multi(ok, p, p, sc, 2, 2, 0, 16, B.UQ_FMT_I8, p, p, p + 16, None, None) == B.UQ_ERR_BAD_ARG  # out alignment
    # uq_encode_decode: the checks of the encoders and of uq_decode
    assert lib.uq_encode_decode(ok, p, p, 127, None, 0, None, 0, 0, 24, B.UQ_FMT_I8, p, p, None, None) == B.UQ_ERR_BAD_ARG   # rng_bits
    assert lib.uq_encode_decode(ok, p, p, 128, None, 0, None, 0, 0, 16, B.UQ_FMT_I8, p, p, None, None) == B.UQ_ERR_BAD_ARG   # s > 127
    assert lib.uq_encode_decode(ok, p, p, 127, None, 0, None, 0, 0, 16, B.UQ_FMT_I8, p, None, None, None) == B.UQ_ERR_BAD_ARG  # out
    assert lib.uq_encode_decode(ok, p, p, 127, sc, 2, None, 2, 0, 16, B.UQ_FMT_I8, p, p, None, None) == B.UQ_ERR_BAD_ARG     # idx
    assert lib.uq_encode_decode(ok, p, p, 127, sc, 2, p, 3, 0, 16, B.UQ_FMT_I8, p, p, None, None) == B.UQ_ERR_BAD_ARG        # idx_bits
    assert lib.uq_index_min(p, 0, 64, 64, 2, p, None) == B.UQ_ERR_BAD_ARG                    # R
    assert lib.uq_index_min(p, 2, 64, 62, 2, p, None) == B.UQ_ERR_BAD_ARG                    # whole words
    assert lib.uq_index_min(p, 2, 32, 64, 2, p, None) == B.UQ_ERR_BAD_ARG                    # rows overlap
    assert lib.uq_index_min(p, 2, 64, 64, 3, p, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode_rows(ok, None, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode_rows(ok, rows, 9, p, 127, None, 0, None, 0, p, None, None) == B.UQ_ERR_BAD_ARG
    rows[1] = p + 1
    assert lib.uq_decode_rows(ok, rows, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode_update(ok, p, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p, None, F(float("nan")), F(0), F(0), None,
                                None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_decode_update(ok, p, B.UQ_FMT_I8, p, 127, None, 0, None, 0, p + 4, None, F(0.1), F(0), F(0), None,
                                None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_randk_gather(ok, p, 1001, 0, p, p, 1024, None, None) == B.UQ_ERR_BAD_ARG     # K > d
    assert lib.uq_randk_gather(ok, p, 10, 0, p, p, 40, None, None) == B.UQ_ERR_BAD_ARG         # stride % 32
    assert lib.uq_randk_gather(ok, p, 10, 0, p, p, 0, None, None) == B.UQ_ERR_BAD_ARG          # stride < K
    assert lib.uq_randk_scatter(100, 101, p, p, p, None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_randk_update(100, 10, p, None, p, F(0.1), None, None) == B.UQ_ERR_BAD_ARG
    assert lib.uq_randk_update(100, 10, p, p, p, F(float("nan")), None, None) == B.UQ_ERR_BAD_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", tmp_path / "missing.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()


def test_a_tensor_on_another_device_is_refused_before_any_launch():
    """The calls launch on the current device's current stream; the binding refuses, on the host,
    a tensor that lives elsewhere (checked here on the rule itself: no GPU, no launch)."""
    B.require_current_device(0, 0)
    B.require_current_device(3, 3, "g")
    for index, current in ((1, 0), (0, 1), (None, 0)):
        with pytest.raises(ValueError, match="current device"):
            B.require_current_device(index, current, "g")
