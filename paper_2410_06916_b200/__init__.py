"""SWIFT self-speculative decoding hot path for one B200 (sm_100a): Python binding over the C library."""
from .binding import (SwiftError, SwiftModel, GenParams, GenStats, lib, load_library, MAX_ROWS, gemm_static, STATIC_SCRATCH_BYTES, LayerSetOptimizer, many_row_schedule)  # noqa: F401
