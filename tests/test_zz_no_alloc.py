"""swift_gemm_static: the GEMM entry point for callers that may not allocate device memory.

Such callers exist wherever this library is a guest: a plug-in inside a serving process that owns the
CUDA allocator and passes in finished tensors, or code running at a moment when cudaMalloc's implicit
synchronisation is not tolerable.  The entry point keeps its split-K scratch in an array compiled into
the library, so the only device memory involved is what the caller passes in.  This file is collected
last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

import synth
from oracle import swift_oracle as so

pytestmark = pytest.mark.gpu


def _model_and_weight(dtype):
    from paper_2410_06916_b200 import SwiftModel
    cfg = synth.ModelConfig("noalloc", n_blocks=1, d_model=1032, n_heads=9, n_kv_heads=3, head_dim=64, ffn=1392,
                            vocab=500, dtype=dtype, seed=31, n_planted=0)
    g = SwiftModel(cfg, max_positions=64)
    w = synth.make_tensor(cfg, "wo", 0, planted=False)          # [d_model, n_heads*head_dim] = [1032, 576]: ragged in N and K
    g.pack("wo", 0, w)
    return cfg, g, w


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_gemm_matches_the_context_gemm_twice_in_a_row(dtype):
    from paper_2410_06916_b200 import gemm_static
    cfg, g, w = _model_and_weight(dtype)
    try:
        w_dev = w.cuda()
        gen = torch.Generator().manual_seed(5)
        # two calls back to back, the second with fewer rows and other data: nothing of the first may survive in it
        for rows in (13, 3):
            x = torch.randn(rows, w.shape[1], generator=gen)
            ref = g.gemm(1, 0, x.numpy())                        # existing entry point (o_proj of block 0)
            x_dev, y_dev = x.cuda(), torch.full((rows, w.shape[0]), float("nan"), device="cuda")
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            gemm_static(w_dev, x_dev, y_dev)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before      # the call made no torch allocation either
            got = y_dev.cpu().numpy()
            scale = float(np.sqrt((ref ** 2).mean()))
            assert np.isfinite(got).all()
            assert np.abs(got - ref).max() < 2e-4 * scale, float(np.abs(got - ref).max() / scale)
            # ... and against the plain fp64 product, so that a defect both entry points share cannot hide
            exact = so.linear(x, w).numpy()
            assert np.abs(got - exact).max() < 2e-4 * scale, float(np.abs(got - exact).max() / scale)
    finally:
        g.close()


def test_static_scratch_gemm_rejects_what_does_not_fit():
    from paper_2410_06916_b200 import SwiftError, gemm_static, STATIC_SCRATCH_BYTES
    N, K = 40000, 2048                                           # 4 splits * 16 * 40000 * 4 bytes = 10.24 MB > 8 MiB
    assert 4 * 16 * N * 4 + 1024 > STATIC_SCRATCH_BYTES
    w = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    x = torch.zeros(2, K, device="cuda")
    y = torch.full((2, N), 7.0, device="cuda")
    with pytest.raises(SwiftError, match="ECAPACITY.*scratch"):
        gemm_static(w, x, y)
    torch.cuda.synchronize()
    assert float(y.min()) == 7.0                                 # nothing was enqueued
    with pytest.raises(SwiftError, match="ECAPACITY"):
        gemm_static(w[:64], torch.zeros(17, K, device="cuda"), torch.zeros(17, 64, device="cuda"))
