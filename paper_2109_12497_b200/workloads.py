"""Seeded synthetic gradient workloads.

This module only makes inputs: shapes, segment tables and random gradient values.  It holds
none of the quantizer's arithmetic and is the one module that both the CUDA tests/benchmark and
the CPU oracle's tests use, so that both sides see bit-identical inputs.  numpy only.

The five workloads stand in for the gradients of the paper's CIFAR10 ResNet50 / VGG16 runs
(Section "Experiments"), which need a dataset and a training loop; here the value distributions
and layer structure are stated recipes:

  c1  single-scale, M=2,  d=2^20 fp32,  N(0, 0.01^2), one segment, s=127, int8 levels,
      scale = max|g| over both workers
  c2  single-scale, M=8,  d=25,557,032 fp32 in 161 layer segments (many small, a few large),
      per-layer std log-uniform in [1e-5, 1e-1] shared by the workers, s=127, int8
  c3  multi-scale on the data of c2, scale set {127 * 8^k, k<4}, 2-bit shared index
  c4  single-scale, M=16, d=2^26 fp32, 1e-3 * Student-t(3), one segment, s=7, two levels per byte
  c5  multi-scale, M=8, d=335,141,888 bf16, N(0, 0.02^2) with 1% of the coordinates x100
      (same coordinates on every worker), 25 MiB buckets, scale set {127 * 8^k, k<8}, 4-bit index

c1 to c4 draw 32 random bits per coordinate (``rng_bits``, 23 of them used), the library's default;
c5 draws 16: its encoder moves only 3.5 bytes per coordinate and worker and is bound by arithmetic,
not by memory, with 32-bit draws (measured: 0.65 of the copy peak, ALU and multiply pipes the
busiest units; the fp32 encoders reach 0.77 to 0.82).  Both widths are tested and timed on every
workload.

``scaled(name, d)`` gives the same recipe at a smaller d for tests.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Optional, Tuple

import numpy as np

F32, BF16 = "f32", "bf16"
NORM_LINF, NORM_L2 = "linf", "l2"
STRIDE_ALIGN = 32  # worker stride is padded to a multiple of this many coordinates


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    quantizer: str            # "single" | "multi"
    M: int
    d: int
    dtype: str                # F32 | BF16
    values: str               # "normal" | "layers" | "student_t3" | "normal_outliers"
    segments: str             # "one" | "layers161" | "buckets25MiB"
    s: int                    # levels of the (smallest) scale
    scales: Tuple[int, ...]   # ascending scale set; (s,) for single-scale
    fmt: str                  # "i8" | "i4x2" | "i2x4" | "i6p"
    idx_bits: int             # 0 for single-scale
    norm: str
    seed: int                 # seed of the quantizer's random draws
    data_seed: int
    rng_bits: int = 32        # width of the random draw per coordinate (16 or 32 Philox bits)
    nseg_hint: int = 1
    bucket_elems: int = 0

    @property
    def stride(self) -> int:
        return -(-self.d // STRIDE_ALIGN) * STRIDE_ALIGN

    @property
    def in_bytes(self) -> int:
        return self.M * self.d * (4 if self.dtype == F32 else 2)


def _geom(s: int, ratio: int, n: int) -> Tuple[int, ...]:
    return tuple(s * ratio ** k for k in range(n))


WORKLOADS = {
    "c1": Workload("c1", "single", 2, 1 << 20, F32, "normal", "one", 127, (127,), "i8", 0,
                   NORM_LINF, 0, 1001),
    "c2": Workload("c2", "single", 8, 25_557_032, F32, "layers", "layers161", 127, (127,), "i8", 0,
                   NORM_L2, 0, 1002, nseg_hint=161),
    "c3": Workload("c3", "multi", 8, 25_557_032, F32, "layers", "layers161", 127,
                   _geom(127, 8, 4), "i8", 2, NORM_L2, 0, 1002, nseg_hint=161),
    "c4": Workload("c4", "single", 16, 1 << 26, F32, "student_t3", "one", 7, (7,), "i4x2", 0,
                   NORM_L2, 0, 1004),
    "c5": Workload("c5", "multi", 8, 335_141_888, BF16, "normal_outliers", "buckets25MiB", 127,
                   _geom(127, 8, 8), "i8", 4, NORM_L2, 0, 1005, rng_bits=16,
                   bucket_elems=25 * (1 << 20) // 2),
}


def scaled(name: str, d: int, M: Optional[int] = None, **overrides) -> Workload:
    """The recipe of workload ``name`` at a smaller size (tests)."""
    w = WORKLOADS[name]
    changes = dict(d=d, name=f"{name}@{d}")
    if M is not None:
        changes["M"] = M
    if w.segments == "buckets25MiB":
        # keep several whole buckets plus a ragged last one
        changes["bucket_elems"] = max(64, d // 5 + 3)
    changes.update(overrides)
    return dataclasses.replace(w, **changes)


# ---------------------------------------------------------------------------------------------
# segment tables
# ---------------------------------------------------------------------------------------------

def layer_sizes(d: int, nseg: int, seed: int) -> np.ndarray:
    """nseg positive sizes summing to d: about two thirds small tensors (norm scales, biases)
    and one third large ones (convolution / linear weights), in shuffled order."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x5E6]))
    n_small = (nseg * 2) // 3
    n_big = nseg - n_small
    small = rng.integers(64, 2049, size=n_small).astype(np.float64)
    big = np.exp(rng.uniform(np.log(4096.0), np.log(2.4e6), size=n_big))
    if small.sum() > d / 4:                    # tiny test sizes: shrink the small tensors
        small *= (d / 4) / small.sum()
    big *= (d - small.sum()) / big.sum()
    sizes = np.maximum(1, np.floor(np.concatenate([small, big]))).astype(np.int64)
    rng.shuffle(sizes)
    sizes[np.argmax(sizes)] += d - sizes.sum()  # remainder goes to the largest tensor
    assert sizes.sum() == d and (sizes > 0).all()
    return sizes


def segment_offsets(w: Workload) -> np.ndarray:
    """int64 offsets, length nseg+1, first 0 and last d."""
    if w.segments == "one":
        return np.array([0, w.d], dtype=np.int64)
    if w.segments == "layers161":
        nseg = min(w.nseg_hint, max(1, w.d // 8))
        sizes = layer_sizes(w.d, nseg, w.data_seed)
        return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    if w.segments == "buckets25MiB":
        edges = list(range(0, w.d, w.bucket_elems)) + [w.d]
        return np.array(edges, dtype=np.int64)
    raise ValueError(w.segments)


# ---------------------------------------------------------------------------------------------
# values
# ---------------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


_CHUNK = 1 << 22


def _layer_std(w: Workload, seg_off: np.ndarray) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[w.data_seed, 0x57D]))
    return (10.0 ** rng.uniform(-5.0, -1.0, size=len(seg_off) - 1)).astype(np.float32)


def _outlier_chunk(w: Workload, c0: int, n: int) -> np.ndarray:
    """Bernoulli(0.01) mask of coordinates c0..c0+n-1, the same for every worker."""
    rng = np.random.Generator(np.random.Philox(key=[w.data_seed, 0x0071], counter=[0, 0, 0, c0]))
    return rng.random(n, dtype=np.float32) < np.float32(0.01)


def _fill_worker(w: Workload, m: int, row: np.ndarray, seg_off: np.ndarray, std: np.ndarray) -> None:
    """Write worker m's d values into row[:d] (float32 array, or uint16 bf16 bits)."""
    for c0 in range(0, w.d, _CHUNK):
        n = min(_CHUNK, w.d - c0)
        # one generator per (worker, chunk): the values do not depend on how chunks are threaded
        rng = np.random.Generator(np.random.Philox(key=[w.data_seed, m + 1], counter=[0, 0, 0, c0]))
        if w.values == "normal":
            x = rng.standard_normal(n, dtype=np.float32) * np.float32(0.01)
        elif w.values == "layers":
            x = rng.standard_normal(n, dtype=np.float32)
            j = np.searchsorted(seg_off, np.arange(c0, c0 + n), side="right") - 1
            x *= std[np.minimum(j, len(std) - 1)]
        elif w.values == "student_t3":
            z = rng.standard_normal((4, n), dtype=np.float32)
            chi = (z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / np.float32(3.0)
            x = np.float32(1e-3) * z[0] / np.sqrt(np.maximum(chi, np.float32(1e-30)))
        elif w.values == "normal_outliers":
            x = rng.standard_normal(n, dtype=np.float32) * np.float32(0.02)
            x[_outlier_chunk(w, c0, n)] *= np.float32(100.0)
        else:
            raise ValueError(w.values)
        if w.dtype == F32:
            row[c0:c0 + n] = x
        else:
            row[c0:c0 + n] = f32_to_bf16_bits(x)


def generate(w: Workload, out: Optional[np.ndarray] = None, threads: int = 8, workers=None) -> np.ndarray:
    """Gradients of all workers as an [M, stride] array (float32, or uint16 holding bf16 bits);
    columns d..stride-1 are zero padding.  ``out`` may be a preallocated (e.g. pinned) buffer.
    ``workers`` (a sequence of worker numbers) makes only those workers' rows, in that order: a
    process that holds part of the job's workers gets exactly the rows the whole array has."""
    np_dtype = np.float32 if w.dtype == F32 else np.uint16
    rows = list(range(w.M)) if workers is None else [int(m) for m in workers]
    if out is None:
        out = np.zeros((len(rows), w.stride), dtype=np_dtype)
    assert out.shape == (len(rows), w.stride) and out.dtype == np_dtype
    out[:, w.d:] = 0
    seg_off = segment_offsets(w)
    std = _layer_std(w, seg_off) if w.values == "layers" else None
    with ThreadPoolExecutor(max_workers=max(1, threads)) as pool:
        list(pool.map(lambda k: _fill_worker(w, rows[k], out[k], seg_off, std), range(len(rows))))
    return out
