"""The allocation-free attention-importance entry point, for callers that cannot allocate device
memory (fixed-pool hosts, real-time loops, code that only receives raw pointers).

Collected last on purpose.  The call must give the same scores as the workspace-taking entry point
on two calls in a row (the built-in scratch keeps the first call's contents, which must not leak
into the second), and must refuse sizes beyond its built-in scratch.
"""
import numpy as np
import pytest
import torch

from paper_2603_00198_b200 import binding, inputs
from util_gpu import dev, score_rel_err

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_workspace_variant_twice():
    ctx = binding.Context(0)
    try:
        cases = [("bf16", 3000, 100, 8, 2, 128, 2, 71), ("f32", 777, 33, 4, 4, 64, 1, 72)]
        for dtype, n_vis, M, Hq, Hkv, d, Bz, seed in cases:      # second call: other shape, other data
            a = inputs.attn_score_inputs(seed, n_vis + M, Hq, Hkv, d, dtype, batch=Bz)
            q, k = dev(a["q"], dtype), dev(a["k"], dtype)
            scale = 1.0 / np.sqrt(d)
            ref = binding.str_attn_importance(ctx, q, k, n_vis, M, scale)
            out = torch.full((Bz, n_vis), float("nan"), dtype=torch.float32, device="cuda")
            binding.str_attn_importance_static(ctx, q, k, n_vis, M, scale, out=out)
            ctx.check_status()
            got, ref = out.cpu().numpy(), ref.cpu().numpy()
            assert np.all(np.isfinite(got))
            assert score_rel_err(got, ref) <= 1e-3
            assert abs(got[0].astype(np.float64).sum() - 1.0) < 1e-4
    finally:
        ctx.close()


def test_static_scratch_variant_rejects_oversize_requests():
    ctx = binding.Context(0)
    try:
        Hq, M = 64, binding.STR_ATTN_STATIC_MAX_ROWS // 64 + 1      # Bz*Hq*M just beyond the limit
        q = torch.zeros((1, 8 + M, Hq, 16), dtype=torch.bfloat16, device="cuda")
        k = torch.zeros((1, 8 + M, 1, 16), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(binding.StrError) as e:
            binding.str_attn_importance_static(ctx, q, k, 8, M, 1.0)
        assert e.value.code == -3
    finally:
        ctx.close()
