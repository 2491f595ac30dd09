"""uq — all-reduce-compatible unbiased gradient quantizers, hand-written CUDA for B200 (sm_100a).

``binding`` exposes the C ABI of ``include/uq.h`` one to one; ``workloads`` makes the seeded
synthetic gradients; ``build`` compiles the library in-tree with nvcc.
"""
from .binding import (  # noqa: F401
    Layout, UqError, lib, uq_version,
    uq_agree_scale, uq_agree_scale_static, uq_encode_single, uq_select_scale_multi, uq_encode_multi, uq_aggregate, uq_decode, uq_decode_update,
    uq_randk_gather, uq_randk_scatter, uq_randk_update, uq_index_min, uq_decode_rows, uq_select_encode_multi, uq_step,
    UQ_F32, UQ_BF16, UQ_NORM_LINF, UQ_NORM_L2, UQ_FMT_I8, UQ_FMT_I4X2, UQ_FMT_I2X4, UQ_FMT_I6P, UQ_SRC_LEVELS, UQ_SRC_SUMS,
    UQ_STATUS_NONFINITE, UQ_STATUS_BAD_SEGMENTS, UQ_STATUS_SCALE_OVERFLOW, UQ_STATUS_BAD_INDEX,
)
