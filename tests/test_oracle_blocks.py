"""CPU pins for the block glue around the recurrence.  The paper does not define these pieces,
so they are pinned to textbook definitions, library routines and brute force on tiny inputs."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle


def test_bf16_rounding_mirror():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -3.140625, 0.0, 1e-3])
    r = oracle.round_to_bf16(v)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == 1.0 + 2 ** -6
    assert r[4] == -3.140625 and r[5] == 0.0 and abs(r[6] - 1e-3) < 1e-3 * 2 ** -8
    np.testing.assert_array_equal(oracle.round_to_bf16(r), r)


def test_rmsnorm_softplus_silu():
    r = np.random.default_rng(0)
    u = r.normal(size=(5, 64)) * 7
    y = oracle.rmsnorm(u, eps=0.0)
    np.testing.assert_allclose((y * y).mean(axis=1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(y / y[:, :1], u / u[:, :1], rtol=1e-12)
    v = np.array([-30.0, -1.0, 0.0, 2.0, 40.0])
    np.testing.assert_allclose(oracle.softplus(v), np.log1p(np.exp(v)), rtol=1e-12)
    np.testing.assert_allclose(oracle.silu(v), v * (1 / (1 + np.exp(-v))), rtol=1e-12)


def test_causal_conv_matches_library_convolution():
    r = np.random.default_rng(1)
    T, Cc, W = 11, 3, 4
    v, w, b = r.normal(size=(T, Cc)), r.normal(size=(Cc, W)), r.normal(size=Cc)
    out = oracle.causal_conv1d_silu(v, w, b)
    for c in range(Cc):
        pre = np.convolve(v[:, c], w[c, ::-1])[:T] + b[c]     # last tap multiplies the current token
        np.testing.assert_allclose(out[:, c], oracle.silu(pre), rtol=1e-12)
    # causal: the first output sees only the first input through the last tap
    np.testing.assert_allclose(out[0], oracle.silu(b + w[:, -1] * v[0]), rtol=1e-12)


def test_rope_is_a_rotation_with_relative_phase():
    r = np.random.default_rng(2)
    d, theta = 8, 1.0e6
    q, k = r.normal(size=(1, 1, d)), r.normal(size=(1, 1, d))
    np.testing.assert_allclose(oracle.rope(q, [0], theta), q, rtol=1e-15)
    dots = []
    for pm, pi in ((5, 2), (105, 102), (40003, 40000)):
        qr, kr = oracle.rope(q, [pm], theta), oracle.rope(k, [pi], theta)
        np.testing.assert_allclose(np.linalg.norm(qr), np.linalg.norm(q), rtol=1e-12)
        dots.append(float((qr * kr).sum()))
    np.testing.assert_allclose(dots, dots[0], rtol=1e-9)
    # pair (0, d/2) turns by exactly pos radians (frequency theta^0 = 1)
    e = np.zeros((1, 1, d)); e[0, 0, 0] = 1.0
    out = oracle.rope(e, [0.5], theta)
    np.testing.assert_allclose([out[0, 0, 0], out[0, 0, d // 2]], [np.cos(0.5), np.sin(0.5)], rtol=1e-12)


def test_attention_forward_brute_force_and_special_cases():
    r = np.random.default_rng(3)
    T, Hq, Hkv, d = 9, 4, 2, 3
    q, k, v = r.normal(size=(T, Hq, d)), r.normal(size=(T, Hkv, d)), r.normal(size=(T, Hkv, d))
    o = oracle.attention_forward(q, k, v, 0.7, slab=4)
    for h in range(Hq):
        kv = h // 2
        for t in range(T):
            w = softmax(np.array([np.dot(q[t, h], k[j, kv]) * 0.7 for j in range(t + 1)]))
            np.testing.assert_allclose(o[t, h], sum(w[j] * v[j, kv] for j in range(t + 1)), rtol=1e-11)
    o0 = oracle.attention_forward(np.zeros_like(q), k, v, 0.7)
    np.testing.assert_allclose(o0[:, 0], np.cumsum(v[:, 0], axis=0) / np.arange(1, T + 1)[:, None], rtol=1e-12)


def test_attention_rows_is_the_same_definition_row_by_row():
    r = np.random.default_rng(6)
    T, Hq, Hkv, d = 23, 6, 3, 5
    q, k, v = r.normal(size=(T, Hq, d)), r.normal(size=(T, Hkv, d)), r.normal(size=(T, Hkv, d))
    rows = [0, 1, 7, 22]
    o = oracle.attention_rows(q, k, v, 0.9, rows)
    np.testing.assert_allclose(o, oracle.attention_forward(q, k, v, 0.9)[rows], atol=1e-13)
    for i, t in enumerate(rows):                 # a library softmax over the allowed keys
        for h in range(Hq):
            w = softmax((k[:t + 1, h // 2] @ q[t, h]) * 0.9)
            np.testing.assert_allclose(o[i, h], w @ v[:t + 1, h // 2], atol=1e-13)


def test_stack_identity_schedule_and_text_rows_last():
    from paper_2603_00198_b200 import inputs
    ms = dict(D=32, H=4, p=8, n=8, G=2, Q=16, conv=4)
    at = dict(D=32, Hq=4, Hkv=2, d=8, theta=1.0e6)
    layers = inputs.stack_params(5, "MAM", ms, at, "f32")
    n_vis, M = 24, 4
    h0 = inputs.hidden_inputs(5, n_vis + M, 32, "f32")[0]
    full, pos, idx, _ = oracle.stack_prefill(h0, M, layers, [n_vis] * 3)
    assert full.shape == h0.shape and list(idx) == list(range(n_vis + M))
    K = oracle.schedule_keep_counts([10000, 5000, 2500], n_vis, 0)
    red, pos, idx, trace = oracle.stack_prefill(h0, M, layers, K)
    assert K == [24, 12, 6] and red.shape == (6 + M, 32)
    assert list(idx[-M:]) == list(range(n_vis, n_vis + M)) and np.all(np.diff(idx) > 0)
    assert np.array_equal(pos, idx)
    assert trace[0]["kept"] is None and len(trace[1]["kept"]) == 12 and len(trace[2]["kept"]) == 6
    np.testing.assert_allclose(trace[1]["scores"].sum(), 1.0, rtol=1e-12)   # layer 2 is attention


def test_ffn_block_textbook_cases():
    # the paper names FFN blocks without defining them; these pin the restatement to its own definition
    r = np.random.default_rng(7)
    D, F, T = 6, 10, 5
    u = r.normal(size=(T, D))
    prm = dict(D=D, F=F, W_up=r.normal(size=(D, F)), W_down=r.normal(size=(F, D)))
    out = oracle.ffn_block(u, prm)
    ref = np.zeros_like(u)
    for t in range(T):                                   # explicit loops
        nrm = u[t] / np.sqrt(np.mean(u[t] ** 2) + 1e-5)
        hid = [max(sum(nrm[i] * prm["W_up"][i, f] for i in range(D)), 0.0) ** 2 for f in range(F)]
        ref[t] = u[t] + [sum(hid[f] * prm["W_down"][f, j] for f in range(F)) for j in range(D)]
    np.testing.assert_allclose(out, ref, rtol=1e-12)
    # a zero down-projection leaves the residual stream alone; negating the up-projection of a row with all
    # positive pre-activations switches the block off for it; scaling W_up by 2 scales the update by 4
    np.testing.assert_array_equal(oracle.ffn_block(u, dict(prm, W_down=np.zeros((F, D)))), u)
    pos_up = np.abs(prm["W_up"])
    u_pos = np.abs(u)
    np.testing.assert_allclose(oracle.ffn_block(u_pos, dict(prm, W_up=-pos_up)), u_pos, rtol=1e-13)
    np.testing.assert_allclose(oracle.ffn_block(u, dict(prm, W_up=2 * prm["W_up"])) - u, 4 * (out - u), rtol=1e-12)


def test_stack_with_ffn_layers_keeps_the_row_set():
    from paper_2603_00198_b200 import inputs
    ms = dict(D=32, H=4, p=8, n=8, G=2, Q=16, conv=4)
    at = dict(D=32, Hq=4, Hkv=2, d=8, theta=1.0e6)
    layers = inputs.stack_params(6, "MFAF", ms, at, "f32", ffn_dim=48)
    n_vis, M = 24, 4
    h0 = inputs.hidden_inputs(6, n_vis + M, 32, "f32")[0]
    out, pos, idx, trace = oracle.stack_prefill(h0, M, layers, [12, 12, 6, 6])
    assert out.shape == (6 + M, 32) and trace[1]["kept"] is None and trace[3]["kept"] is None
    assert len(trace[0]["kept"]) == 12 and len(trace[2]["kept"]) == 6
    # an FFN layer acts row by row: running it on the compacted rows equals compacting its output
    h1, _ = oracle.mamba2_block(h0, layers[0][1])
    rows = np.concatenate([trace[0]["kept"], np.arange(n_vis, n_vis + M)])
    np.testing.assert_allclose(oracle.ffn_block(h1[rows], layers[1][1]), oracle.ffn_block(h1, layers[1][1])[rows], rtol=1e-13)
    with pytest.raises(AssertionError):
        oracle.stack_prefill(h0, M, layers, [12, 6, 6, 6])          # an FFN layer may not reduce


def test_attn_block_rows_and_resumed_stack_agree_with_the_whole_computation():
    """Two conveniences of the oracle used by the large GPU parity tests: the attention block evaluated for a few
    rows only, and a stack continued from a reduced context (carried ids passed in) with its trace of layer
    inputs.  Both must reproduce the plain whole-sequence run."""
    from paper_2603_00198_b200 import inputs
    ms = dict(D=32, H=4, p=8, n=8, G=2, Q=16, conv=4)
    at = dict(D=32, Hq=4, Hkv=2, d=8, theta=1.0e6)
    layers = inputs.stack_params(15, "MAMA", ms, at, "f32")
    n_vis, M = 40, 6
    h0 = inputs.hidden_inputs(15, n_vis + M, 32, "f32")[0]
    pos = np.arange(n_vis + M) * 3 + 1                          # arbitrary ascending positions
    full, mid = oracle.attn_block(h0, pos, layers[1][1])
    rows = [0, 5, 17, n_vis + M - 1]
    part, mid_r = oracle.attn_block_rows(h0, pos, layers[1][1], rows)
    np.testing.assert_allclose(part, full[rows], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(mid_r["k"], mid["k"], rtol=0, atol=0)
    # whole run with a trace of layer inputs; layers 2.. re-run from the stored input of layer 2 give the same result
    K = [n_vis, 20, 20, 10]
    out, opos, oidx, trace = oracle.stack_prefill(h0, M, layers, K, keep_inputs=True)
    rec = trace[2]
    assert rec["n_in"] == 20 and rec["hidden_in"].shape == (20 + M, 32)
    out2, pos2, idx2, trace2 = oracle.stack_prefill(rec["hidden_in"], M, layers[2:], K[2:], positions=rec["positions_in"],
                                                    idx_map=rec["idx_map_in"])
    np.testing.assert_array_equal(out2, out)
    np.testing.assert_array_equal(idx2, oidx)
    np.testing.assert_array_equal(pos2, opos)
    # hand-off records: a Mamba layer's final state is the recurrence's, an attention layer's keys are those of the
    # rows that leave it, with their original positions
    assert trace[0]["final_state"].shape == (4, 8, 8) and trace[1]["k"].shape == (20 + M, 2, 8)
    np.testing.assert_array_equal(trace[1]["kv_positions"], trace[2]["positions_in"])
    np.testing.assert_array_equal(trace[3]["kv_positions"], opos)
