"""GPU parity for the block glue (GEMM, norms, conv/split, RoPE, causal GQA attention) against the
oracle's textbook definitions."""
import numpy as np
import pytest

import oracle
from paper_2603_00198_b200 import binding, inputs
from util_gpu import dev, host, max_rel_err

pytestmark = pytest.mark.gpu
TOL = {"bf16": 2e-2, "f32": 2e-4}


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.check_status()
    c.close()


@pytest.mark.parametrize("dtype,M,N,K", [("bf16", 300, 200, 256), ("f32", 65, 130, 70), ("bf16", 1056, 1184, 256),
                                         ("bf16", 4224, 1024, 4096), ("bf16", 128, 18560, 4096), ("f32", 1, 7, 3),
                                         ("bf16", 257, 136, 8192)])
def test_gemm_with_residual(ctx, dtype, M, N, K):
    g = inputs.rng(51, M + N + K)
    a = inputs.to_grid(g.standard_normal((M, K), dtype=np.float32), dtype)
    w = inputs.to_grid(g.standard_normal((N, K), dtype=np.float32) / np.sqrt(K), dtype)
    r = inputs.to_grid(g.standard_normal((M, N), dtype=np.float32), dtype)
    ref = a.astype(np.float64) @ w.astype(np.float64).T
    got = host(binding.str_gemm(ctx, dev(a, dtype), dev(w, dtype)))
    assert max_rel_err(got, ref) <= TOL[dtype]
    got = host(binding.str_gemm(ctx, dev(a, dtype), dev(w, dtype), residual=dev(r, dtype)))
    assert max_rel_err(got, ref + r) <= TOL[dtype]


@pytest.mark.parametrize("M,N,K", [(129, 256, 64), (300, 200, 256), (1056, 1184, 256), (257, 136, 8192), (8320, 2304, 1024)])
def test_gemm_on_cta_pairs_is_bit_identical_to_the_lone_cta_kernel(M, N, K, monkeypatch):
    """Above 128 rows the GEMM runs on CTA pairs (one 256-row MMA per K-slice across two SMs); a context created with
    STR_GEMM_PAIR=0 keeps the one-CTA kernel.  Same K order, same epilogue arithmetic: the outputs must be equal bit
    for bit, with and without the residual, on ragged M, N and K."""
    g = inputs.rng(57, M + N + K)
    a = dev(inputs.to_grid(g.standard_normal((M, K), dtype=np.float32), "bf16"), "bf16")
    w = dev(inputs.to_grid(g.standard_normal((N, K), dtype=np.float32) / np.sqrt(K), "bf16"), "bf16")
    r = dev(inputs.to_grid(g.standard_normal((M, N), dtype=np.float32), "bf16"), "bf16")
    outs = []
    for flag in ("0", "1"):
        monkeypatch.setenv("STR_GEMM_PAIR", flag)
        c = binding.Context(0)
        outs.append((binding.str_gemm(c, a, w), binding.str_gemm(c, a, w, residual=r)))
        c.check_status()
        assert c.path_counts() == (2, 0)
        c.close()
    assert bool((outs[0][0] == outs[1][0]).all()) and bool((outs[0][1] == outs[1][1]).all())


@pytest.mark.parametrize("dtype,rows,D", [("bf16", 100, 4096), ("f32", 33, 256), ("bf16", 5, 40), ("bf16", 9, 8192),
                                          ("bf16", 3, 36)])
def test_rmsnorm(ctx, dtype, rows, D):
    u = inputs.hidden_inputs(52, rows, D, dtype)[0] * 3.0
    u = inputs.to_grid(u, dtype)
    got = host(binding.str_rmsnorm(ctx, dev(u, dtype)))
    assert max_rel_err(got, oracle.rmsnorm(u)) <= TOL[dtype]


@pytest.mark.parametrize("dtype,Bz,T,H,p,n,G", [("bf16", 1, 300, 16, 64, 128, 2), ("f32", 2, 70, 8, 32, 16, 1),
                                                ("bf16", 3, 70, 8, 64, 64, 1), ("bf16", 2, 33, 4, 16, 32, 2),
                                                ("bf16", 1, 2, 8, 64, 128, 8), ("bf16", 2, 33000, 8, 8, 8, 1),
                                                ("f32", 1, 66000, 2, 4, 4, 1)])
def test_conv_split_and_gated_norm(ctx, dtype, Bz, T, H, p, n, G):
    d_inner, gn = H * p, G * n
    ld = 2 * d_inner + 2 * gn + H
    g = inputs.rng(53, T)
    z = inputs.to_grid(g.standard_normal((Bz * T, ld), dtype=np.float32), dtype)
    cw = g.uniform(-0.5, 0.5, size=(d_inner + 2 * gn, 4)).astype(np.float32)
    cb = g.uniform(-0.1, 0.1, size=(d_inner + 2 * gn,)).astype(np.float32)
    dtb = inputs.softplus_inverse(g.uniform(1e-3, 1e-1, size=H)).astype(np.float32)
    x, Bm, Cm, dt = binding.str_mamba_conv_split(ctx, dev(z, dtype), dev(cw), dev(cb), dev(dtb), Bz, T, H, p, n, G)
    for b in range(Bz):
        zz = z[b * T:(b + 1) * T].astype(np.float64)
        ref = oracle.causal_conv1d_silu(zz[:, d_inner:2 * d_inner + 2 * gn], cw, cb)     # per sequence: no leak across b
        assert max_rel_err(host(x)[b].reshape(T, d_inner), ref[:, :d_inner]) <= TOL[dtype]
        assert max_rel_err(host(Bm)[b].reshape(T, gn), ref[:, d_inner:d_inner + gn]) <= TOL[dtype]
        assert max_rel_err(host(Cm)[b].reshape(T, gn), ref[:, d_inner + gn:]) <= TOL[dtype]
        rdt = oracle.softplus(zz[:, 2 * d_inner + 2 * gn:] + dtb[None, :])
        assert np.abs(host(dt)[b] / rdt - 1).max() <= 1e-5
    y = inputs.to_grid(g.standard_normal((Bz * T, d_inner), dtype=np.float32), dtype)
    got = host(binding.str_gated_rmsnorm(ctx, dev(y, dtype), dev(z, dtype), d_inner))
    ref = oracle.rmsnorm(y.astype(np.float64) * oracle.silu(z[:, :d_inner].astype(np.float64)))
    assert max_rel_err(got, ref) <= TOL[dtype]


@pytest.mark.parametrize("dtype,Bz,T,D,H,p,n,G", [("bf16", 1, 4224, 512, 8, 64, 128, 2), ("bf16", 3, 333, 256, 8, 32, 32, 1),
                                                  ("bf16", 1, 100, 256, 8, 64, 128, 2), ("bf16", 4, 31, 128, 16, 64, 64, 1),
                                                  ("bf16", 2, 1, 128, 8, 32, 32, 1), ("f32", 2, 70, 64, 8, 32, 16, 1),
                                                  ("bf16", 1, 300, 256, 4, 16, 8, 1)])
def test_in_projection_with_the_prescan_step_in_its_epilogue(ctx, dtype, Bz, T, D, H, p, n, G):
    """str_mamba_in_proj_conv against the two calls it stands for (str_gemm, str_mamba_conv_split): every output equal
    bit for bit, whether the conv ran in the projection's epilogue (the first five cases: sequences that start and end
    inside a warp's 32 rows, fewer rows than one tile, one-token sequences) or the call composed the two kernels."""
    d_inner, gn = H * p, G * n
    N = 2 * d_inner + 2 * gn + H
    g = inputs.rng(58, T + D)
    u = dev(inputs.to_grid(g.standard_normal((Bz * T, D), dtype=np.float32), dtype), dtype)
    w = dev(inputs.to_grid(g.standard_normal((N, D), dtype=np.float32) / np.sqrt(D), dtype), dtype)
    cw = dev(g.uniform(-0.5, 0.5, size=(d_inner + 2 * gn, 4)).astype(np.float32))
    cb = dev(g.uniform(-0.1, 0.1, size=(d_inner + 2 * gn,)).astype(np.float32))
    dtb = dev(inputs.softplus_inverse(g.uniform(1e-3, 1e-1, size=H)).astype(np.float32))
    zx = binding.str_gemm(ctx, u, w)
    ref = binding.str_mamba_conv_split(ctx, zx, cw, cb, dtb, Bz, T, H, p, n, G)
    got = binding.str_mamba_in_proj_conv(ctx, u, w, cw, cb, dtb, Bz, T, H, p, n, G)
    ctx.check_status()
    assert bool((got[0][:, :d_inner] == zx[:, :d_inner]).all())                 # the gate columns
    for a, b, name in zip(got[1:], ref, "xBCd"):
        assert bool((a == b).all()), name


# the last case has more than 65535 rows (batch 4 of the 16512-token attention layers has 66048)
@pytest.mark.parametrize("dtype,Bz,T,Hq,Hkv,d", [("bf16", 1, 200, 8, 2, 128), ("f32", 2, 50, 4, 4, 32),
                                                   ("bf16", 2, 35000, 2, 1, 16)])
def test_rope_split(ctx, dtype, Bz, T, Hq, Hkv, d):
    g = inputs.rng(54, T)
    qkv = inputs.to_grid(g.standard_normal((Bz * T, (Hq + 2 * Hkv) * d), dtype=np.float32), dtype)
    pos = np.sort(g.choice(70000, size=(Bz, T)), axis=1).astype(np.int32)      # carried original positions
    q, k, v = binding.str_rope_split(ctx, dev(qkv, dtype), dev(pos), Bz, T, Hq, Hkv, d, 1.0e6)
    for b in range(Bz):
        blk = qkv[b * T:(b + 1) * T].astype(np.float64)
        rq = oracle.rope(blk[:, :Hq * d].reshape(T, Hq, d), pos[b], 1.0e6)
        rk = oracle.rope(blk[:, Hq * d:(Hq + Hkv) * d].reshape(T, Hkv, d), pos[b], 1.0e6)
        tol = 1e-2 if dtype == "bf16" else 1e-5
        assert max_rel_err(host(q)[b], rq) <= tol and max_rel_err(host(k)[b], rk) <= tol
        assert np.array_equal(host(v)[b].reshape(T, -1), blk[:, (Hq + Hkv) * d:])


@pytest.mark.parametrize("dtype,Bz,T,Hq,Hkv,d", [("bf16", 1, 700, 8, 2, 128), ("f32", 2, 130, 4, 2, 32),
                                                   ("bf16", 1, 64, 2, 1, 64), ("f32", 1, 1, 2, 2, 16),
                                                   # head_dim 128 in bf16 runs on the tensor cores: tile edges,
                                                   # ragged tails, one query-tile pair and several, no GQA, batch
                                                   ("bf16", 1, 1, 2, 1, 128), ("bf16", 1, 128, 2, 2, 128),
                                                   ("bf16", 1, 129, 4, 1, 128), ("bf16", 2, 256, 2, 1, 128),
                                                   ("bf16", 1, 257, 2, 2, 128), ("bf16", 2, 1000, 4, 2, 128),
                                                   ("bf16", 1, 1536, 4, 4, 128)])
def test_attention_forward(ctx, dtype, Bz, T, Hq, Hkv, d):
    g = inputs.rng(55, T)
    q = inputs.to_grid(g.standard_normal((Bz, T, Hq, d), dtype=np.float32), dtype)
    k = inputs.to_grid(g.standard_normal((Bz, T, Hkv, d), dtype=np.float32), dtype)
    v = inputs.to_grid(g.standard_normal((Bz, T, Hkv, d), dtype=np.float32), dtype)
    scale = 1.0 / np.sqrt(d)
    o = host(binding.str_attn_prefill(ctx, dev(q, dtype), dev(k, dtype), dev(v, dtype), scale))
    for b in range(Bz):
        assert max_rel_err(o[b], oracle.attention_forward(q[b], k[b], v[b], scale)) <= TOL[dtype]


def test_attention_forward_growing_logits_rescale(ctx):
    """Logits that keep growing along the key axis force the running row maximum up tile after tile, so
    the accumulator rescaling path runs many times; a second input has one huge late key."""
    T, Hq, Hkv, d = 900, 2, 1, 128
    g = inputs.rng(56, T)
    q = inputs.to_grid(g.standard_normal((1, T, Hq, d), dtype=np.float32), "bf16")
    k = inputs.to_grid(g.standard_normal((1, T, Hkv, d), dtype=np.float32), "bf16")
    v = inputs.to_grid(g.standard_normal((1, T, Hkv, d), dtype=np.float32), "bf16")
    u = g.standard_normal(d).astype(np.float32)
    u /= np.linalg.norm(u)
    ramp = (np.arange(T, dtype=np.float32) / T * 60.0)[:, None, None]
    q2 = inputs.to_grid(q + 4.0 * u, "bf16")
    k2 = inputs.to_grid(k + ramp * u, "bf16")               # q.k grows by ~240/sqrt(d)*... along the keys
    k3 = k.copy()
    k3[0, 700] = inputs.to_grid(40.0 * u, "bf16")           # one dominant key late in the sequence
    scale = 1.0 / np.sqrt(d)
    for kk in (k2, k3):
        o = host(binding.str_attn_prefill(ctx, dev(q2, "bf16"), dev(kk, "bf16"), dev(v, "bf16"), scale))
        assert np.all(np.isfinite(o))
        assert max_rel_err(o[0], oracle.attention_forward(q2[0], kk[0], v[0], scale)) <= TOL["bf16"]


@pytest.mark.parametrize("dtype,n", [("bf16", 8 * 1000), ("bf16", 1003), ("f32", 777), ("bf16", 8)])
def test_relu_squared(ctx, dtype, n):
    v = inputs.to_grid(inputs.hidden_inputs(57, 1, n, dtype)[0] * 2.0, dtype)
    ref = np.maximum(v.astype(np.float64), 0.0) ** 2
    x = dev(v, dtype)
    assert max_rel_err(host(binding.str_relu_squared(ctx, x)), ref) <= TOL[dtype]
    binding.str_relu_squared(ctx, x, inplace=True)
    assert max_rel_err(host(x), ref) <= TOL[dtype]


@pytest.mark.parametrize("dtype,Bz,T,Hq,Hkv,d,keep", [("bf16", 2, 1500, 4, 2, 128, 0.25), ("bf16", 1, 700, 8, 2, 128, 0.1),
                                                      ("f32", 1, 333, 4, 4, 32, 0.3), ("bf16", 2, 450, 4, 2, 64, 0.5)])
def test_attention_for_a_gathered_subset_of_query_rows(ctx, dtype, Bz, T, Hq, Hkv, d, keep):
    """A layer that selects before its attention only needs the surviving rows' outputs: computed for a gathered
    subset (ascending indices into the key sequence) they equal the oracle's rows and are bit-identical to the rows
    of the full call, whatever other rows share their tile."""
    import torch
    g = inputs.rng(31, T)
    q = inputs.to_grid(g.standard_normal((Bz, T, Hq, d), dtype=np.float32), dtype)
    k = inputs.to_grid(g.standard_normal((Bz, T, Hkv, d), dtype=np.float32) * 1.5, dtype)
    v = inputs.to_grid(g.standard_normal((Bz, T, Hkv, d), dtype=np.float32), dtype)
    n_text = 20
    n_keep = int((T - n_text) * keep)
    rows = np.stack([np.concatenate([np.sort(g.choice(T - n_text, size=n_keep, replace=False)), np.arange(T - n_text, T)])
                     for _ in range(Bz)]).astype(np.int32)
    scale = 1.0 / np.sqrt(d)
    full = binding.str_attn_prefill(ctx, dev(q, dtype), dev(k, dtype), dev(v, dtype), scale)
    qr = np.stack([q[b][rows[b]] for b in range(Bz)])
    part = binding.str_attn_prefill_rows(ctx, dev(qr, dtype), dev(rows), dev(k, dtype), dev(v, dtype), scale)
    ctx.check_status()
    for b in range(Bz):
        assert bool((part[b] == full[b][torch.from_numpy(rows[b]).long().cuda()]).all())
        sample = [0, 1, n_keep // 2, n_keep - 1, n_keep, n_keep + n_text - 1]
        ref = oracle.attention_rows(q[b], k[b], v[b], scale, [int(rows[b][j]) for j in sample])
        assert max_rel_err(host(part)[b][sample], ref) <= (2e-2 if dtype == "bf16" else 2e-4)
