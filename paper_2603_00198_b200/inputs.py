"""Seeded synthetic inputs shaped like the paper's long-video workloads.

Host-side numpy only: no CUDA, no method arithmetic.  Both the GPU path and the CPU oracle are
fed from here so that they see bit-identical values.  Arrays come back as float32 whose values
already sit on the grid of the requested storage type ("bf16" or "f32"), so the GPU side can
narrow them without further rounding and the oracle can widen them to fp64 exactly.

Recipe (visual tokens first, text query last, as in Section 3.1 of the paper):
  hidden states ~ N(0,1); projection weights ~ N(0, 1/d_model);
  A_h = -exp(U(ln 1, ln 16)) per head; dt = softplus(raw + dt_bias) with
  dt_bias = softplus^-1(U(1e-3, 1e-1)); scan-level tests draw dt ~ U(1e-3, 1e-1) directly;
  depthwise conv taps ~ U(-1/2, 1/2) (width 4), conv bias ~ U(-0.1, 0.1).
"""
import numpy as np

# Workload shapes.  C0..C4 follow the five benchmark configurations: a tiny fp32 Mamba-2 layer,
# an 8B-class Mamba-2 layer, a GQA attention layer, the 12-layer hybrid stack, and the sweep.
MAMBA_TINY = dict(D=256, H=8, p=32, n=16, G=1, Q=64, conv=4)
MAMBA_8B = dict(D=4096, H=128, p=64, n=128, G=8, Q=256, conv=4)
ATTN_8B = dict(D=4096, Hq=32, Hkv=8, d=128, theta=1.0e6)

CONFIGS = {
    "C0": dict(kind="mamba", shape=MAMBA_TINY, dtype="f32", seed=0, n_vis=1024, n_text=32, keep_bp=2500),
    "C1": dict(kind="mamba", shape=MAMBA_8B, dtype="bf16", seed=1, n_vis=4096, n_text=128, keep_bp=2500),
    "C2": dict(kind="attn", shape=ATTN_8B, dtype="bf16", seed=2, n_vis=16384, n_text=128, keep_bp=2500),
    "C3": dict(kind="stack", pattern="MMMMMA" * 2, mamba=MAMBA_8B, attn=ATTN_8B, dtype="bf16", seed=3,
               n_vis=32768, n_text=128,
               alpha_bp=[10000] * 4 + [5000] * 4 + [2500] * 4, min_keep=256),
}


def rng(seed, stream=0):
    """Counter-based generator: one independent stream per (seed, stream)."""
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def to_grid(a, dtype):
    """Round float values onto the storage grid of ``dtype`` and return float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype != "bf16":
        raise ValueError(dtype)
    u = a.view(np.uint32)
    u = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).reshape(a.shape)


def bf16_bits(a):
    """uint16 bit patterns of float32 values that already sit on the bf16 grid."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def ssd_inputs(seed, T, H, p, n, G, dtype, batch=1):
    """Scan-level inputs: x [Bz,T,H,p], dt [Bz,T,H] fp32, A [H] fp32, B,C [Bz,T,G,n]."""
    g = rng(seed, 1)
    x = to_grid(g.standard_normal((batch, T, H, p), dtype=np.float32), dtype)
    Bm = to_grid(g.standard_normal((batch, T, G, n), dtype=np.float32), dtype)
    Cm = to_grid(g.standard_normal((batch, T, G, n), dtype=np.float32), dtype)
    dt = g.uniform(1e-3, 1e-1, size=(batch, T, H)).astype(np.float32)
    A = (-np.exp(g.uniform(0.0, np.log(16.0), size=H))).astype(np.float32)
    return dict(x=x, dt=dt, A=A, B=Bm, C=Cm)


def attn_score_inputs(seed, T, Hq, Hkv, d, dtype, batch=1):
    """Post-RoPE q [Bz,T,Hq,d] and k [Bz,T,Hkv,d] with unit-variance entries."""
    g = rng(seed, 2)
    q = to_grid(g.standard_normal((batch, T, Hq, d), dtype=np.float32), dtype)
    k = to_grid(g.standard_normal((batch, T, Hkv, d), dtype=np.float32), dtype)
    return dict(q=q, k=k)


def hidden_inputs(seed, T, D, dtype, batch=1):
    g = rng(seed, 3)
    return to_grid(g.standard_normal((batch, T, D), dtype=np.float32), dtype)


def score_vectors(seed, n, kind="uniform", batch=1):
    """Non-negative fp32 score rows for selection tests.

    kinds: uniform | heavy (a fifth of 256-token frames carry most of the mass, as the paper's
    sparsity analysis describes) | ties (few distinct values) | equal | ascending | descending.
    """
    g = rng(seed, 4)
    if kind == "uniform":
        s = g.uniform(0.0, 1.0, size=(batch, n))
    elif kind == "heavy":
        s = g.uniform(0.0, 1.0, size=(batch, n)) * 1e-2
        frames = max(1, n // 256)
        for b in range(batch):
            hot = g.choice(frames, size=max(1, frames // 5), replace=False)
            for f in hot:
                s[b, f * 256:(f + 1) * 256] += g.exponential(1.0, size=len(s[b, f * 256:(f + 1) * 256]))
    elif kind == "ties":
        s = g.integers(0, 7, size=(batch, n)).astype(np.float64) * 0.125
    elif kind == "equal":
        s = np.full((batch, n), 0.5)
    elif kind == "ascending":
        s = np.tile(np.arange(n, dtype=np.float64) / max(1, n), (batch, 1))
    elif kind == "descending":
        s = np.tile(np.arange(n, 0, -1, dtype=np.float64) / max(1, n), (batch, 1))
    else:
        raise ValueError(kind)
    return s.astype(np.float32)


def softplus_inverse(v):
    v = np.asarray(v, dtype=np.float64)
    return v + np.log(-np.expm1(-v))


def mamba_layer_params(seed, layer, shape, dtype):
    """Random-init Mamba-2 block parameters.  W_in [D, 2*d_inner + 2*G*n + H] maps the normed
    hidden state to [z | x B C | dt_raw]; W_out [d_inner, D]."""
    D, H, p, n, G, W = shape["D"], shape["H"], shape["p"], shape["n"], shape["G"], shape["conv"]
    d_inner = H * p
    d_in_proj = 2 * d_inner + 2 * G * n + H
    g = rng(seed, 100 + layer)
    std = 1.0 / np.sqrt(D)
    prm = dict(H=H, p=p, n=n, G=G, D=D)
    prm["W_in"] = to_grid(g.standard_normal((D, d_in_proj), dtype=np.float32) * std, dtype)
    prm["W_out"] = to_grid(g.standard_normal((d_inner, D), dtype=np.float32) * std, dtype)
    prm["conv_w"] = g.uniform(-0.5, 0.5, size=(d_inner + 2 * G * n, W)).astype(np.float32)
    prm["conv_b"] = g.uniform(-0.1, 0.1, size=(d_inner + 2 * G * n,)).astype(np.float32)
    prm["A"] = (-np.exp(g.uniform(0.0, np.log(16.0), size=H))).astype(np.float32)
    prm["dt_bias"] = softplus_inverse(g.uniform(1e-3, 1e-1, size=H)).astype(np.float32)
    return prm


def attn_layer_params(seed, layer, shape, dtype):
    """Random-init GQA block parameters.  W_qkv [D, (Hq+2*Hkv)*d] = [q | k | v]; W_o [Hq*d, D]."""
    D, Hq, Hkv, d = shape["D"], shape["Hq"], shape["Hkv"], shape["d"]
    g = rng(seed, 100 + layer)
    std = 1.0 / np.sqrt(D)
    prm = dict(Hq=Hq, Hkv=Hkv, d=d, D=D, theta=float(shape["theta"]))
    prm["W_qkv"] = to_grid(g.standard_normal((D, (Hq + 2 * Hkv) * d), dtype=np.float32) * std, dtype)
    prm["W_o"] = to_grid(g.standard_normal((Hq * d, D), dtype=np.float32) * std, dtype)
    return prm


def ffn_layer_params(seed, layer, D, F, dtype):
    """Random-init FFN block parameters.  W_up [D, F], W_down [F, D]; the down projection is scaled so that the
    block's output stays O(1) after the squared activation."""
    g = rng(seed, 200 + layer)
    prm = dict(D=D, F=F)
    prm["W_up"] = to_grid(g.standard_normal((D, F), dtype=np.float32) / np.sqrt(D), dtype)
    prm["W_down"] = to_grid(g.standard_normal((F, D), dtype=np.float32) / np.sqrt(3.0 * F), dtype)
    return prm


def stack_params(seed, pattern, mamba_shape, attn_shape, dtype, ffn_dim=0):
    layers = []
    for l, kind in enumerate(pattern):
        if kind == "M":
            layers.append(("M", mamba_layer_params(seed, l, mamba_shape, dtype)))
        elif kind == "A":
            layers.append(("A", attn_layer_params(seed, l, attn_shape, dtype)))
        elif kind == "F":
            D = (mamba_shape or attn_shape)["D"]
            layers.append(("F", ffn_layer_params(seed, l, D, ffn_dim or 4 * D, dtype)))
        else:
            raise ValueError(kind)
    return layers


def sweep_alpha_bp(final_bp, n_layers=12):
    """Three equal low-to-high stages 100% -> sqrt(final) -> final, in basis points
    (reproduces 100/50/25 for a 25% final budget)."""
    mid = int(np.floor(np.sqrt(final_bp / 10000.0) * 10000.0 + 1e-9))
    third = n_layers // 3
    return [10000] * third + [mid] * third + [int(final_bp)] * (n_layers - 2 * third)
