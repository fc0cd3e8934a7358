"""GPU parity at the benchmark configurations' full layer widths (8B-class Mamba-2 layer: d_model 4096, 128 heads of
64, state 128, 8 groups; GQA attention layer: 32 query / 8 KV heads of 128), i.e. on the tensor-core kernels the
benchmark times, against the fp64 oracle with the bf16 storage mirror.

  * C1 as a layer, C2 as a layer (whole output on a short sequence, sampled rows + the full score vector at 16384+128).
  * The C3 layer pattern [M,M,M,M,M,A]x2 with the 100/50/25 schedule on a shorter sequence, TEACHER-FORCED per layer:
    GPU layer l is fed the oracle's input of layer l (hidden states and carried token ids), so exactly one layer's
    arithmetic separates the two and the MAXIMUM row error can be asserted in every layer; batch 1 and batch 4.
  * The decoder hand-off (final Mamba states, keys / values / positions of the rows leaving attention layers).

Layer-level tolerances (derived in the design notes): outputs max|err| / max|ref| <= 2e-2 on the rows both sides keep;
scores <= 3e-3 relative (both sides round the projections to bf16 at the same points, but fp32 against fp64
accumulation flips single bf16 roundings of B, C, q, k elements); kept sets equal up to swaps among tokens whose
oracle scores lie within that same 3e-3 of the threshold; carried ids bit-exact given the selection.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_00198_b200 import binding, inputs
from util_gpu import SCORE_TOL, assert_kept_matches, check_layer, check_stack_teacher_forced, dev, host

pytestmark = pytest.mark.gpu
MS, AT = inputs.MAMBA_8B, inputs.ATTN_8B
RND = oracle.round_to_bf16


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.check_status()
    c.close()


def test_c1_mamba_layer_at_full_width(ctx):
    cfg = inputs.CONFIGS["C1"]
    n_vis, M = cfg["n_vis"], cfg["n_text"]
    K = oracle.schedule_keep_counts([cfg["keep_bp"]], n_vis, 0)
    assert K == [1024] == binding.str_schedule_keep_counts([cfg["keep_bp"]], n_vis, 0)
    layers = inputs.stack_params(cfg["seed"], "M", MS, AT, "bf16")
    h0 = inputs.hidden_inputs(cfg["seed"], n_vis + M, MS["D"], "bf16")
    ref, rpos, ridx, trace = oracle.stack_prefill(h0[0], M, layers, K, RND)
    ids = np.arange(n_vis + M, dtype=np.int32)[None]
    check_layer(ctx, layers[0], 1, n_vis, M, K[0], h0, ids, ids, [ref], [ridx], [trace[0]], Q=MS["Q"])


def test_c2_attention_layer_at_full_width_whole_output(ctx):
    n_vis, M = 2048, 128
    layers = inputs.stack_params(2, "A", MS, AT, "bf16")
    h0 = inputs.hidden_inputs(2, n_vis + M, AT["D"], "bf16")
    K = [n_vis // 4]
    ref, rpos, ridx, trace = oracle.stack_prefill(h0[0], M, layers, K, RND)
    ids = np.arange(n_vis + M, dtype=np.int32)[None]
    check_layer(ctx, layers[0], 1, n_vis, M, K[0], h0, ids, ids, [ref], [ridx], [trace[0]])
    assert abs(trace[0]["scores"].sum() - 1.0) < 1e-9


def test_c2_attention_layer_at_full_length_sampled_rows(ctx):
    cfg = inputs.CONFIGS["C2"]
    n_vis, M = cfg["n_vis"], cfg["n_text"]                            # 16384 + 128
    T = n_vis + M
    K = n_vis * cfg["keep_bp"] // 10000
    layers = inputs.stack_params(cfg["seed"], "A", MS, AT, "bf16")
    prm = layers[0][1]
    h0 = inputs.hidden_inputs(cfg["seed"], T, AT["D"], "bf16")
    # the oracle's projections, scores and selection for every token; its attention output for sampled kept rows
    g = inputs.rng(cfg["seed"], 77)
    mid = oracle.attn_block_projections(h0[0], np.arange(T), prm, RND)
    s_ref = oracle.attn_importance(mid["q"], mid["k"], n_vis, M, mid["scale"])
    kept_ref = oracle.topk_select(s_ref, K)
    st = binding.Stack(ctx, layers, "bf16", 1, n_vis, M, [K])
    out, pos, idx, tr = binding.str_stack_prefill(st, dev(h0, "bf16"), want_trace=True)
    ctx.check_status()
    s_gpu, kept = tr[0]["scores"][0].cpu().numpy(), tr[0]["kept"][0].cpu().numpy()
    assert abs(float(s_gpu.astype(np.float64).sum()) - 1.0) < 1e-4
    assert np.abs(s_gpu / s_ref - 1).max() <= SCORE_TOL
    assert_kept_matches(kept, kept_ref, s_ref, tol=SCORE_TOL)
    gi = idx[0].cpu().numpy()
    assert np.array_equal(gi[:K], kept) and np.array_equal(gi[K:], np.arange(n_vis, T))
    both = np.intersect1d(kept, kept_ref)
    rows = np.unique(np.concatenate([g.choice(both, size=12, replace=False), [both[0], both[-1], T - M, T - 1]]))
    ref_rows, _ = oracle.attn_block_rows(h0[0], np.arange(T), prm, rows, RND, mid=mid)
    where = np.searchsorted(gi, rows)
    assert np.array_equal(gi[where], rows)
    got = host(out)[0][where]
    assert np.abs(got - ref_rows).max() / np.abs(ref_rows).max() <= 2e-2


@pytest.fixture(scope="module")
def c3_layers():
    cfg = inputs.CONFIGS["C3"]
    return cfg, inputs.stack_params(cfg["seed"], cfg["pattern"], MS, AT, "bf16")


@pytest.mark.parametrize("Bz,n_vis,seed", [(1, 2048, 3), (4, 384, 4)])
def test_c3_layer_pattern_teacher_forced_at_full_width(ctx, c3_layers, Bz, n_vis, seed):
    """[M,M,M,M,M,A]x2 at full width, 100/50/25: every layer against the oracle's own input of that layer.  The
    batch-4 case draws its hidden states from the sweep configuration's seed."""
    cfg, layers = c3_layers
    M = cfg["n_text"]
    K = oracle.schedule_keep_counts(cfg["alpha_bp"], n_vis, 0)
    assert K == binding.str_schedule_keep_counts(cfg["alpha_bp"], n_vis, 0) == [n_vis] * 4 + [n_vis // 2] * 4 + [n_vis // 4] * 4
    h0 = inputs.hidden_inputs(seed, n_vis + M, MS["D"], "bf16", batch=Bz)
    # Against the oracle's free-running output only the bookkeeping is compared at this width: rounding differences
    # compound through twelve random-init layers (median row difference 6e-2) and any near-tie swap changes the rows
    # after it; the per-layer bounds and the composition identity inside the helper are the statement about accuracy.
    worst, (out, gpos, gidx, tr), runs = check_stack_teacher_forced(ctx, layers, "bf16", Bz, n_vis, M, K, h0, Q=MS["Q"])
    print("max row error per layer:", " ".join("%.1e" % w for w in worst))
    for b in range(Bz):
        assert len(np.intersect1d(gidx[b].cpu().numpy(), runs[b][2])) >= 0.9 * gidx.shape[1]
    assert bool(torch.isfinite(out.float()).all())


def test_decoder_hand_off_of_the_reduced_context(ctx):
    """What a decoder takes over after the reduced prefill: each Mamba layer's final state (the dropped tokens stay
    absorbed in it) and, per attention layer, keys / values / original positions of the rows that leave the layer."""
    ms = dict(D=512, H=8, p=64, n=128, G=2, Q=128, conv=4)
    at = dict(D=512, Hq=4, Hkv=2, d=128, theta=1.0e6)
    n_vis, M = 640, 32
    layers = inputs.stack_params(91, "MAMA", ms, at, "bf16")
    h0 = inputs.hidden_inputs(91, n_vis + M, 512, "bf16")
    K = [n_vis, n_vis // 2, n_vis // 2, n_vis // 4]            # the attention layers (1 and 3) reduce
    ref, rpos, ridx, trace = oracle.stack_prefill(h0[0], M, layers, K, RND, keep_inputs=True)
    st = binding.Stack(ctx, layers, "bf16", 1, n_vis, M, K, Q=128)
    res = binding.str_stack_prefill_ex(st, dev(h0, "bf16"), want_handoff=True, want_trace=True)
    ctx.check_status()
    plain = binding.str_stack_prefill(st, dev(h0, "bf16"))
    assert bool((plain[0] == res["hidden"]).all()) and bool((plain[2] == res["idx_map"]).all())
    # layer 0 (Mamba) and layer 1 (attention) see the same tokens on both sides
    (l0, fs0), (l2, fs2) = res["mamba_final_states"]
    assert (l0, l2) == (0, 2) and fs0.shape == (1, 8, 64, 128)
    f_ref = trace[0]["final_state"]
    assert np.abs(fs0[0].cpu().numpy() - f_ref).max() / np.abs(f_ref).max() <= 1e-2
    (l1, k1), (l3, k3) = res["attn_k"]
    (_, v1), (_, v3) = res["attn_v"]
    (_, p1), (_, p3) = res["attn_pos"]
    assert (l1, l3) == (1, 3) and k1.shape == (1, K[1] + M, 2, 128) and k3.shape == (1, K[3] + M, 2, 128)
    kept1 = res["trace"][0]["kept"][0].cpu().numpy()
    assert_kept_matches(kept1, trace[1]["kept"], trace[1]["scores"], tol=SCORE_TOL)
    gp1 = p1[0].cpu().numpy()
    assert np.array_equal(gp1[:K[1]], kept1) and np.array_equal(gp1[K[1]:], np.arange(n_vis, n_vis + M))
    common, a, c = np.intersect1d(gp1, trace[1]["kv_positions"], return_indices=True)
    assert len(common) >= 0.98 * len(gp1)
    for got, want in ((k1, trace[1]["k"]), (v1, trace[1]["v"])):
        g_ = host(got)[0][a]
        assert np.abs(g_ - want[c]).max() / np.abs(want).max() <= 2e-2
    # the last layer's rows are the rows of the final output
    assert np.array_equal(p3[0].cpu().numpy(), res["positions"][0].cpu().numpy())
    assert bool(torch.isfinite(fs2).all()) and bool(torch.isfinite(k3.float()).all()) and bool(torch.isfinite(v3.float()).all())
