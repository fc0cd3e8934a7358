"""The allocation-free attention-importance entry point, for callers that cannot allocate device
memory (fixed-pool hosts, real-time loops, code that only receives raw pointers).

Collected last on purpose.  The call must give the oracle's scores (and those of the workspace-taking entry point)
on two calls in a row (the built-in scratch keeps the first call's contents, which must not leak into the
second), must leave the device's free memory untouched, must work at exactly its size limit and refuse sizes
beyond it.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_00198_b200 import binding, inputs
from util_gpu import dev, score_rel_err

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_oracle_and_workspace_variant_twice():
    ctx = binding.Context(0)
    try:
        cases = [("bf16", 3000, 100, 8, 2, 128, 2, 71), ("f32", 777, 33, 4, 4, 64, 1, 72)]
        for dtype, n_vis, M, Hq, Hkv, d, Bz, seed in cases:      # second call: other shape, other data
            a = inputs.attn_score_inputs(seed, n_vis + M, Hq, Hkv, d, dtype, batch=Bz)
            q, k = dev(a["q"], dtype), dev(a["k"], dtype)
            scale = 1.0 / np.sqrt(d)
            ref_ws = binding.str_attn_importance(ctx, q, k, n_vis, M, scale)
            out = torch.full((Bz, n_vis), float("nan"), dtype=torch.float32, device="cuda")
            binding.str_attn_importance_static(ctx, q, k, n_vis, M, scale, out=out)      # first call on the device: set-up
            torch.cuda.synchronize()
            # the property the entry point exists for: with a caller-owned output, a call moves no device memory
            free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
            binding.str_attn_importance_static(ctx, q, k, n_vis, M, scale, out=out)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
            ctx.check_status()
            got = out.cpu().numpy()
            assert np.all(np.isfinite(got))
            assert score_rel_err(got, ref_ws.cpu().numpy()) <= 1e-3
            for b in range(Bz):
                ref = oracle.attn_importance(a["q"][b], a["k"][b], n_vis, M, scale)
                assert score_rel_err(got[b], ref) <= 1e-3
                assert abs(got[b].astype(np.float64).sum() - 1.0) < 1e-4
    finally:
        ctx.close()


def test_static_scratch_variant_at_exactly_its_limit():
    """Bz * Hq * n_text == the built-in scratch: the row sums end at the last float of the array."""
    ctx = binding.Context(0)
    try:
        Hq, M, d, n_vis = 64, binding.STR_ATTN_STATIC_MAX_ROWS // 64, 16, 8
        a = inputs.attn_score_inputs(73, n_vis + M, Hq, 1, d, "bf16")
        q, k = dev(a["q"], "bf16"), dev(a["k"], "bf16")
        ref = binding.str_attn_importance(ctx, q, k, n_vis, M, 0.25).cpu().numpy()
        got = binding.str_attn_importance_static(ctx, q, k, n_vis, M, 0.25).cpu().numpy()
        ctx.check_status()
        assert score_rel_err(got, ref) <= 1e-3 and abs(got[0].astype(np.float64).sum() - 1.0) < 1e-4
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
