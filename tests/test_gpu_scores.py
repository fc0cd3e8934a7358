"""GPU parity: importance scores (attention-layer score, Eq. 2 and the Eq. 1 variant) against the oracle, and the
score -> select pipeline with the swap tolerance."""
import numpy as np
import pytest

import oracle
from paper_2603_00198_b200 import binding, inputs
from util_gpu import assert_kept_matches, dev, score_rel_err

pytestmark = pytest.mark.gpu
SCORE_TOL = 1e-3      # relative, fp32 (stated target)


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.check_status()
    c.close()


MAMBA_CASES = [
    # dtype, n_vis, M, H, n, G, Bz
    ("f32", 1024, 32, 8, 16, 1, 1),          # config 0
    ("bf16", 4096, 128, 128, 128, 8, 1),     # config 1
    ("bf16", 1000, 100, 16, 64, 4, 2),       # ragged tiles, batch
    ("f32", 70, 3, 4, 32, 2, 1),
    ("bf16", 5, 1, 2, 16, 1, 1),
    # d_state 128 in bf16 runs on the tensor cores: text counts that need padding to 16, more than 128 text
    # rows, ragged token tiles, a single token, batch
    ("bf16", 1000, 100, 16, 128, 4, 2),
    ("bf16", 300, 1, 8, 128, 8, 1),
    ("bf16", 777, 200, 32, 128, 2, 1),
    ("bf16", 1, 16, 4, 128, 1, 3),
    ("bf16", 129, 256, 8, 128, 2, 1),
]


@pytest.mark.parametrize("dtype,n_vis,M,H,n,G,Bz", MAMBA_CASES)
def test_mamba_importance_matches_eq2(ctx, dtype, n_vis, M, H, n, G, Bz):
    T = n_vis + M
    d = inputs.ssd_inputs(31, T, H, 16, n, G, dtype, batch=Bz)
    got = binding.str_mamba_importance(ctx, dev(d["B"], dtype), dev(d["C"], dtype), dev(d["dt"]), n_vis, M).cpu().numpy()
    k = max(1, n_vis // 4)
    for b in range(Bz):
        ref = oracle.mamba_importance(d["B"][b], d["C"][b], d["dt"][b], n_vis, M)
        assert score_rel_err(got[b], ref) <= SCORE_TOL
        kept = binding.str_topk_select(ctx, dev(got[b:b + 1]), k).cpu().numpy()[0]
        assert_kept_matches(kept, oracle.topk_select(ref, k), ref)


DYN_CASES = [
    # dtype, n_vis, M, H, n, G, Bz
    ("f32", 1024, 32, 8, 16, 1, 1),          # config 0 shape (plain fp32 kernel)
    ("bf16", 4096, 128, 128, 128, 8, 1),     # config 1 shape: tensor cores, 16 heads per group
    ("bf16", 1000, 100, 16, 128, 4, 2),      # padded text rows, ragged token tiles, 4 heads per group, batch
    ("bf16", 300, 1, 8, 128, 8, 1),          # one text row, one head per group
    ("bf16", 777, 200, 32, 128, 2, 1),       # more than 128 text rows: plain kernel
    ("bf16", 1, 16, 4, 128, 1, 3),
    ("bf16", 70, 3, 4, 32, 2, 1),            # d_state the tensor-core kernel does not tile
    ("bf16", 2500, 64, 42, 128, 2, 1),       # 21 heads per group: 63 of the 64 decay columns in use
]


def _dyn_err(got, ref):
    """Relative error where the oracle's score is within fp32's reach of the largest one; beyond that the
    cumulative decay underflows in fp32 (the oracle, in fp64, still holds 1e-40 and smaller) and the GPU
    value only has to be as negligible."""
    floor = 1e-30 * ref.max()
    big = ref >= floor
    assert np.all(got[~big] <= 2 * floor)
    return score_rel_err(got[big], ref[big]), int(big.sum())


@pytest.mark.parametrize("dtype,n_vis,M,H,n,G,Bz", DYN_CASES)
def test_mamba_full_dynamic_score_matches_eq1(ctx, dtype, n_vis, M, H, n, G, Bz):
    T = n_vis + M
    d = inputs.ssd_inputs(33, T, H, 16, n, G, dtype, batch=Bz)
    got = binding.str_mamba_importance_dynamic(ctx, dev(d["B"], dtype), dev(d["C"], dtype), dev(d["dt"]), dev(d["A"]),
                                               n_vis, M).cpu().numpy()
    ctx.check_status()
    for b in range(Bz):
        ref = oracle.mamba_importance_full_dynamic(d["B"][b], d["C"][b], d["dt"][b], d["A"], n_vis, M)
        err, n_big = _dyn_err(got[b], ref)
        assert err <= SCORE_TOL
        assert np.all(got[b] >= 0) and np.all(np.isfinite(got[b]))
        # selection on this score, with a budget that stays above the underflow floor
        k = max(1, min(n_vis // 4, n_big // 2))
        kept = binding.str_topk_select(ctx, dev(got[b:b + 1]), k).cpu().numpy()[0]
        assert_kept_matches(kept, oracle.topk_select(ref, k), ref)


def test_mamba_full_dynamic_score_without_decay_is_eq2(ctx):
    # A = 0: every Abar is one and the score must fall back to the content alignment of Eq. 2
    n_vis, M, H, n, G = 1500, 96, 32, 128, 4
    d = inputs.ssd_inputs(34, n_vis + M, H, 16, n, G, "bf16")
    B, C, dt = dev(d["B"], "bf16"), dev(d["C"], "bf16"), dev(d["dt"])
    dyn = binding.str_mamba_importance_dynamic(ctx, B, C, dt, dev(np.zeros(H, dtype=np.float32)), n_vis, M).cpu().numpy()[0]
    eq2 = binding.str_mamba_importance(ctx, B, C, dt, n_vis, M).cpu().numpy()[0]
    assert score_rel_err(dyn, eq2) <= 1e-4


ATTN_CASES = [
    # dtype, n_vis, M, Hq, Hkv, d, Bz
    ("bf16", 16384, 128, 32, 8, 128, 1),     # config 2
    ("f32", 1000, 33, 4, 2, 64, 2),
    ("bf16", 300, 5, 6, 2, 32, 1),
    ("f32", 64, 1, 2, 2, 16, 1),
    ("bf16", 3, 2, 4, 1, 128, 1),
    # head_dim 128 in bf16 runs on the tensor cores: padded text counts, more than 128 text rows, ragged key
    # tiles (last 256-key step and last 128-key tile partly beyond the visual keys), no GQA, batch
    ("bf16", 1000, 100, 8, 2, 128, 2),
    ("bf16", 777, 200, 4, 4, 128, 1),
    ("bf16", 129, 256, 2, 1, 128, 1),
    ("bf16", 5000, 1, 8, 8, 128, 1),
    ("bf16", 256, 16, 4, 2, 128, 3),
]


@pytest.mark.parametrize("dtype,n_vis,M,Hq,Hkv,d,Bz", ATTN_CASES)
def test_attn_importance_matches_definition(ctx, dtype, n_vis, M, Hq, Hkv, d, Bz):
    T = n_vis + M
    a = inputs.attn_score_inputs(32, T, Hq, Hkv, d, dtype, batch=Bz)
    scale = 1.0 / np.sqrt(d)
    got = binding.str_attn_importance(ctx, dev(a["q"], dtype), dev(a["k"], dtype), n_vis, M, scale).cpu().numpy()
    k = max(1, n_vis // 4)
    for b in range(Bz):
        ref = oracle.attn_importance(a["q"][b], a["k"][b], n_vis, M, scale)
        assert score_rel_err(got[b], ref) <= SCORE_TOL
        assert abs(got[b].astype(np.float64).sum() - 1.0) < 1e-4          # softmax over the visual keys
        kept = binding.str_topk_select(ctx, dev(got[b:b + 1]), k).cpu().numpy()[0]
        assert_kept_matches(kept, oracle.topk_select(ref, k), ref)


def test_attn_importance_large_logits_stay_finite(ctx):
    a = inputs.attn_score_inputs(33, 200 + 4, 2, 1, 64, "f32")
    a["q"] *= 30.0
    got = binding.str_attn_importance(ctx, dev(a["q"]), dev(a["k"]), 200, 4, 1.0).cpu().numpy()[0]
    ref = oracle.attn_importance(a["q"][0], a["k"][0], 200, 4, 1.0)
    assert np.all(np.isfinite(got)) and abs(got.sum() - 1.0) < 1e-4
    big = ref > 1e-6
    assert score_rel_err(got[big], ref[big]) <= SCORE_TOL


def test_score_argument_validation(ctx):
    d = inputs.ssd_inputs(34, 40, 4, 16, 16, 2, "f32")
    with pytest.raises(binding.StrError):      # n_vis + n_text != T
        binding.str_mamba_importance(ctx, dev(d["B"]), dev(d["C"]), dev(d["dt"]), 30, 5)
    a = inputs.attn_score_inputs(34, 40, 4, 2, 16, "f32")
    with pytest.raises(binding.StrError):
        binding.str_attn_importance(ctx, dev(a["q"]), dev(a["k"]), 41, 0, 1.0)


@pytest.mark.parametrize("dtype,n_vis,M,Hq,Hkv,d,Bz", [
    ("bf16", 16384, 128, 32, 8, 128, 1),     # config 2 shape, tensor cores
    ("bf16", 1000, 100, 8, 2, 128, 2),       # padded text rows, ragged key tiles, batch
    ("bf16", 300, 200, 4, 4, 128, 1),        # more than 128 text rows
    ("f32", 1000, 33, 4, 2, 64, 2),          # plain fp32 path
    ("bf16", 3, 2, 4, 1, 128, 1),            # fewer visual keys than text-visible keys matter most
    ("bf16", 64, 1, 2, 2, 32, 1),
])
def test_attention_importance_causal_row_normaliser(ctx, dtype, n_vis, M, Hq, Hkv, d, Bz):
    T = n_vis + M
    x = inputs.attn_score_inputs(35, T, Hq, Hkv, d, dtype, batch=Bz)
    scale = 1.0 / np.sqrt(d)
    q, k = dev(x["q"], dtype), dev(x["k"], dtype)
    got = binding.str_attn_importance(ctx, q, k, n_vis, M, scale, denominator="causal_row").cpu().numpy()
    vis = binding.str_attn_importance(ctx, q, k, n_vis, M, scale).cpu().numpy()
    ctx.check_status()
    for b in range(Bz):
        ref = oracle.attn_importance(x["q"][b], x["k"][b], n_vis, M, scale, "causal_row")
        assert score_rel_err(got[b], ref) <= SCORE_TOL
        assert got[b].sum() < 1.0 and np.all(got[b] <= vis[b] * (1 + 1e-5))      # some of every row's mass stays on text keys


def test_score_variants_reject_bad_arguments(ctx):
    d = inputs.ssd_inputs(36, 40, 8, 16, 128, 2, "bf16")
    B, C, dt, A = dev(d["B"], "bf16"), dev(d["C"], "bf16"), dev(d["dt"]), dev(d["A"])
    s = binding.SsmScoreShape(1, 40, 8, 128, 2, binding.STR_BF16)
    L = binding.lib()
    import ctypes
    out = dev(np.zeros((1, 32), dtype=np.float32))
    nb = L.str_mamba_importance_dynamic_workspace_size(ctypes.byref(s), 32, 8)
    ws = ctx.workspace(nb)
    args = lambda n_vis, n_text, ws_bytes: (ctx.handle, ctypes.byref(s), n_vis, n_text, binding._p(B), binding._p(C), binding._p(dt),
                                            binding._p(A), binding._p(out), binding._p(ws), ctypes.c_size_t(ws_bytes), binding._stream())
    assert L.str_mamba_importance_dynamic(*args(32, 8, nb)) == 0
    assert L.str_mamba_importance_dynamic(*args(30, 8, nb)) == -1            # n_vis + n_text != T
    assert L.str_mamba_importance_dynamic(*args(32, 8, 16)) == -3            # workspace too small
    x = inputs.attn_score_inputs(36, 40, 4, 2, 128, "bf16")
    q, k = dev(x["q"], "bf16"), dev(x["k"], "bf16")
    with pytest.raises(KeyError):
        binding.str_attn_importance(ctx, q, k, 32, 8, 0.1, denominator="rows")
    sa = binding.AttnScoreShape(1, 40, 4, 2, 128, binding.STR_BF16)
    nb = L.str_attn_importance_workspace_size(ctypes.byref(sa), 32, 8)
    ws = ctx.workspace(nb)
    rc = L.str_attn_importance_ex(ctx.handle, ctypes.byref(sa), 32, 8, binding._p(q), binding._p(k), ctypes.c_float(0.1), 7,
                                  binding._p(out), binding._p(ws), ctypes.c_size_t(nb), binding._stream())
    assert rc == -1                                                            # unknown normaliser
    ctx.check_status()
    # zero visual tokens: nothing to score, nothing written
    assert binding.str_mamba_importance_dynamic(ctx, B[:, 32:], C[:, 32:], dt[:, 32:], A, 0, 8).shape == (1, 0)
