"""TEST INFRASTRUCTURE ONLY -- plain fp64 CPU oracle for the token-reduced prefill
of a hybrid Mamba-2 / attention layer stack.  Never imported by the product path.

Every function is the paper's definition written out in numpy fp64 (a library
matmul / sort may serve as one step); nothing is chunked, fused or reordered
except ``mamba2_chunked``, which exists only to show that the chunked form equals
the sequential recurrence.  Shapes use the paper's notation: M text (query)
tokens, N visual tokens (visual first, text last), H heads, p head dimension,
n state dimension, G groups.

Pin status (tests/test_oracle_*.py, all CPU):
  mamba2_recurrence      pinned  (unrolled double sum of Eq. 1, closed forms)
  mamba2_unrolled        pinned  (geometric-series closed form, one-token case)
  mamba2_chunked         pinned  (equals the recurrence for many chunk sizes)
  mamba_importance       pinned  (explicit loops of Eq. 2, M=G=1 closed form, invariances)
  attn_importance        pinned  (sums to one, zero-query uniform case, scipy softmax)
  topk_select            pinned  (brute force on tiny inputs, threshold property)
  compact                pinned  (bit-exact gather, index-map composition)
  step_schedule / mean_retention / schedule_keep_counts
                         pinned  (the paper's printed compression percentages)
  score_density          pinned  (closed forms: uniform, one-hot, two-level vectors; brute force)
  sigmoid_schedule       parity unpinned: the printed percentages of the sigmoid rows are
                         not reproduced to the printed digit by any indexing of the formula
  rmsnorm, causal_conv1d_silu, rope, attention_forward, attention_rows, mamba2_block, attn_block, attn_block_projections,
  attn_block_rows, stack_prefill
                         parity unpinned by the paper (it does not define the block around the
                         recurrence); pinned only to textbook definitions, library routines
                         and brute force on tiny inputs
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def _clib():
    global _LIB
    if _LIB is None:
        from . import build as _build
        _LIB = ctypes.CDLL(_build.build())
        _LIB.ssm_recurrence_f64.restype = ctypes.c_int
        _LIB.ssm_recurrence_f64.argtypes = [ctypes.c_long] * 5 + [ctypes.c_void_p] * 9
    return _LIB


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


# ----------------------------------------------------------------------------
# storage rounding mirror
# ----------------------------------------------------------------------------
def round_to_bf16(a):
    """Round fp64 values to the nearest bfloat16 (ties to even), returned as fp64.

    Mirrors the places where the GPU path stores an activation in bf16; it is a
    storage format, not part of the method.  Goes through fp32 first, like a GPU
    that accumulates in fp32 and then narrows.
    """
    f = np.ascontiguousarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def _identity(a):
    return a


# ----------------------------------------------------------------------------
# Mamba-2 recurrence (Section 3.1; appendix "State-Space Recurrence")
# ----------------------------------------------------------------------------
def mamba2_recurrence(x, dt, A, B, C, D=None, init_state=None):
    """Sequential recurrence S_t = Abar_t S_{t-1} + x_t (Delta_t b_t)^T, y_t = S_t c_t.

    x [T,H,p], dt [T,H] (>0), A [H] (<0; Abar_t = exp(dt*A)), B,C [T,G,n].
    Returns (y [T,H,p], final state [H,p,n]).  Runs the C loop in ssm_recurrence.c.
    """
    x, dt, A, B, C = _f64(x), _f64(dt), _f64(A), _f64(B), _f64(C)
    T, H, p = x.shape
    G, n = B.shape[1], B.shape[2]
    assert dt.shape == (T, H) and A.shape == (H,) and B.shape == C.shape == (T, G, n)
    Dv = None if D is None else _f64(D)
    S0 = None if init_state is None else _f64(init_state)
    y = np.empty((T, H, p), dtype=np.float64)
    Sf = np.empty((H, p, n), dtype=np.float64)
    rc = _clib().ssm_recurrence_f64(T, H, p, n, G, _ptr(x), _ptr(dt), _ptr(A), _ptr(B), _ptr(C),
                                    _ptr(Dv), _ptr(S0), _ptr(y), _ptr(Sf))
    if rc != 0:
        raise RuntimeError(f"ssm_recurrence_f64 failed: {rc}")
    return y, Sf


def mamba2_unrolled_weights(dt, A, B, C, h):
    """Eq. 1: w[t,j] = (prod_{u=j+1..t} Abar_u) * (Delta_j b_j)^T c_t for head h, j <= t.

    The "Full Mamba Dynamic" weight.  Returns a lower-triangular [T,T] matrix.
    Pure loops; for tiny T only.
    """
    dt, A, B, C = _f64(dt), _f64(A), _f64(B), _f64(C)
    T, H = dt.shape
    G = B.shape[1]
    g = h // (H // G)
    abar = np.exp(dt[:, h] * A[h])
    w = np.zeros((T, T))
    for t in range(T):
        for j in range(t + 1):
            decay = 1.0
            for u in range(j + 1, t + 1):
                decay *= abar[u]
            w[t, j] = decay * float(np.dot(dt[j, h] * B[j, g], C[t, g]))
    return w


def mamba2_unrolled(x, dt, A, B, C):
    """y_t = sum_{j<=t} w[t,j] x_j (the unrolled "attention form" of the recurrence)."""
    x = _f64(x)
    T, H, p = x.shape
    y = np.zeros((T, H, p))
    for h in range(H):
        w = mamba2_unrolled_weights(dt, A, B, C, h)
        y[:, h, :] = w @ x[:, h, :]
    return y


def mamba2_chunked(x, dt, A, B, C, Q):
    """Chunked (block-decomposed) evaluation of the same recurrence, fp64.

    Obtained by splitting the unrolled sum at chunk boundaries: with the in-chunk
    inclusive cumulative log-decay l_t = sum_{u<=t} dt_u A,
      intra:  y_t += sum_{j<=t, same chunk} exp(l_t - l_j) (c_t.b_j) dt_j x_j
      inter:  y_t += exp(l_t) * S_prev c_t
      carry:  S <- exp(l_end) S + sum_j exp(l_end - l_j) dt_j x_j b_j^T
    Exists to show chunked == sequential; the GPU kernels use this decomposition.
    """
    x, dt, A, B, C = _f64(x), _f64(dt), _f64(A), _f64(B), _f64(C)
    T, H, p = x.shape
    G, n = B.shape[1], B.shape[2]
    y = np.zeros((T, H, p))
    S = np.zeros((H, p, n))
    for h in range(H):
        g = h // (H // G)
        Sh = np.zeros((p, n))
        for s in range(0, T, Q):
            e = min(T, s + Q)
            l = np.cumsum(dt[s:e, h] * A[h])
            causal = np.tri(e - s, dtype=bool)
            Lmat = np.exp(np.where(causal, l[:, None] - l[None, :], -np.inf))   # exp(l_t - l_j), j<=t
            CB = C[s:e, g] @ B[s:e, g].T                         # c_t . b_j
            xbar = dt[s:e, h, None] * x[s:e, h]                  # dt_j x_j
            y[s:e, h] = (Lmat * CB) @ xbar + np.exp(l)[:, None] * (C[s:e, g] @ Sh.T)
            w_end = np.exp(l[-1] - l)                            # exp(l_end - l_j)
            Sh = np.exp(l[-1]) * Sh + (w_end[:, None] * xbar).T @ B[s:e, g]
        S[h] = Sh
    return y, S


# ----------------------------------------------------------------------------
# importance scores (Section 3.1)
# ----------------------------------------------------------------------------
def group_mean_dt(dt, G):
    """Delta-bar[i,g] = mean of Delta[i,h] over the H/G heads of group g.

    Reading: Delta is per head while b is per group and Eq. 2 sums over groups.  The group
    mean equals summing each head's own Delta_h |b.c| and normalising by 1/(M*H), because
    Delta > 0 factors out of the absolute value.
    """
    dt = _f64(dt)
    T, H = dt.shape
    return dt.reshape(T, G, H // G).mean(axis=2)


def mamba_importance(B, C, dt, n_vis, n_text):
    """Eq. 2 (Decoupled Content Alignment): s_i = 1/(M G) sum_{m,g} | bbar_i^(g)T c_m^(g) |.

    bbar_i^(g) = Delta-bar_i^(g) b_i^(g); i runs over the first n_vis (visual) rows, m over the
    last n_text (text) rows.  No decay term.  B,C [T,G,n], dt [T,H].  Returns s [n_vis].
    """
    B, C = _f64(B), _f64(C)
    T, G, n = B.shape
    assert n_vis + n_text == T
    dbar = group_mean_dt(dt, G)
    s = np.zeros(n_vis)
    for g in range(G):
        bbar = dbar[:n_vis, g, None] * B[:n_vis, g, :]           # [n_vis, n]
        align = bbar @ C[n_vis:, g, :].T                          # [n_vis, M]
        s += np.abs(align).sum(axis=1)
    return s / (n_text * G)


def mamba_importance_full_dynamic(B, C, dt, A, n_vis, n_text):
    """The "Full Mamba Dynamic" score (Section 3.1, "Why the Full Mamba Dynamic Fails"): |w_{t,i}| of Eq. 1,
    i.e. content alignment times the cumulative decay between visual token i and text position t,

        s_i = 1/(M H) sum_{m,h} | (prod_{u=i+1..t_m} Abar_u^(h)) (Delta_i^(h) b_i^(g(h)))^T c_{t_m}^(g(h)) |,

    t_m = n_vis + m the m-th text row.  The paper names the per-pair quantity |w_{t,j}| and does not spell
    out the aggregation; the mean over the M text positions and the H heads is taken by analogy with Eq. 2
    (the decay is per head, so heads replace groups).  The decay product is written as the exponential of
    a difference of cumulative sums of Delta_u A_h.  B,C [T,G,n], dt [T,H], A [H] (< 0).  Returns s [n_vis].
    """
    B, C, dt, A = _f64(B), _f64(C), _f64(dt), _f64(A)
    T, G, n = B.shape
    H = dt.shape[1]
    assert n_vis + n_text == T and H % G == 0
    L = np.cumsum(dt * A[None, :], axis=0)                        # [T, H]: log of prod_{u<=t} Abar_u
    s = np.zeros(n_vis)
    for h in range(H):
        g = h // (H // G)
        align = (dt[:n_vis, h, None] * B[:n_vis, g, :]) @ C[n_vis:, g, :].T      # [n_vis, M]
        decay = np.exp(L[None, n_vis:, h] - L[:n_vis, None, h])                  # [n_vis, M], all exponents <= 0
        s += np.abs(decay * align).sum(axis=1)
    return s / (n_text * H)


def attn_importance(q, k, n_vis, n_text, scale, denominator="visual"):
    """s_i = 1/(M Hq) sum_{m,h} softmax_i( q_m^(h) . k_i^(kv(h)) * scale ), text -> visual.

    denominator="visual" (the paper's formula): the softmax normalises over the n_vis visual keys only (the
    subscript i), so the scores of one sequence sum to one.  denominator="causal_row": the normaliser is the one
    of the model's own causal attention row, i.e. it also holds the text keys m' <= m, so s_i is the attention
    probability mass text query m really puts on visual token i (the scores then sum to less than one).
    q [T,Hq,d] (last n_text rows used), k [T,Hkv,d]; query head h reads KV head h // (Hq/Hkv).  Returns s [n_vis].
    """
    assert denominator in ("visual", "causal_row")
    q, k = _f64(q), _f64(k)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    assert n_vis + n_text == T and Hq % Hkv == 0
    s = np.zeros(n_vis)
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        logits = (q[n_vis:, h, :] @ k[:, kv, :].T) * scale        # [M, T]
        if denominator == "visual":
            logits = logits[:, :n_vis]
        else:
            for m in range(n_text):
                logits[m, n_vis + m + 1:] = -np.inf               # causal: text query m sees text keys m' <= m
        logits = logits - logits.max(axis=1, keepdims=True)
        e = np.exp(logits)
        s += (e / e.sum(axis=1, keepdims=True))[:, :n_vis].sum(axis=0)
    return s / (n_text * Hq)


# ----------------------------------------------------------------------------
# selection, compaction, schedule (Sections 3.1 "Token Selection", 3.2, appendix schedules)
# ----------------------------------------------------------------------------
def topk_select(scores, k):
    """Indices of the k largest scores, returned in ascending (temporal) order.

    Full sort by (score descending, index ascending): among equal scores the earlier token
    wins (the paper is silent on ties).  Returns int32 [k].
    """
    scores = np.asarray(scores)
    n = scores.shape[0]
    assert 0 <= k <= n
    order = sorted(range(n), key=lambda i: (-float(scores[i]), i))
    return np.array(sorted(order[:k]), dtype=np.int32)


def compact(hidden, positions, idx_map, kept, n_text):
    """Keep the selected visual rows (in the order given) followed by all text rows."""
    hidden = np.asarray(hidden)
    T = hidden.shape[0]
    n_vis = T - n_text
    rows = [int(i) for i in kept] + list(range(n_vis, T))
    out_h = np.stack([hidden[r] for r in rows]) if rows else hidden[:0].copy()
    out_p = np.array([positions[r] for r in rows], dtype=np.int32)
    out_i = np.array([idx_map[r] for r in rows], dtype=np.int32)
    return out_h, out_p, out_i


def step_schedule(L, segments):
    """Per-layer retention alpha (in basis points) from (first_layer, last_layer, alpha_bp)
    segments, inclusive and 0-indexed, as the paper's schedule table writes them."""
    alpha = [None] * L
    for lo, hi, a in segments:
        for l in range(lo, hi + 1):
            alpha[l] = int(a)
    assert all(a is not None for a in alpha)
    return alpha


def sigmoid_schedule(L, k, x0, a_start, a_end):
    """alpha_l = a_end + (a_start - a_end) * sigmoid(k (x0 - l/L)), l = 0..L-1, as fractions."""
    l = np.arange(L, dtype=np.float64)
    return a_end + (a_start - a_end) / (1.0 + np.exp(-k * (x0 - l / L)))


def mean_retention(alpha_bp):
    """The table's "Comp. (%)": mean over layers of the retention ratio, in percent."""
    return sum(alpha_bp) / len(alpha_bp) / 100.0


def schedule_keep_counts(alpha_bp, n0, min_keep, kinds=None):
    """Visual tokens kept AFTER each layer: K_l = min(n_cur, max(min_keep, floor(alpha_l n0))).

    alpha is a fraction of the ORIGINAL visual count n0 (pinned by the printed compression
    percentages); integer arithmetic in basis points; the count never grows.  With ``kinds`` (a
    sequence of "M" / "A" / "F" per layer) FFN layers never reduce: the paper's all-layer schedules
    cut at Mamba and attention layers, so a cut that falls on an FFN layer is taken by the next
    Mamba / attention layer.
    """
    out, n_cur = [], int(n0)
    for l, a in enumerate(alpha_bp):
        k = (int(a) * int(n0)) // 10000
        k = min(n_cur, max(int(min_keep), k))
        if kinds is not None and kinds[l] == "F":
            k = n_cur
        out.append(k)
        n_cur = k
    return out


def score_density(scores, mass_fraction):
    """The sparsity statistic of Section 2 ("tokens needed for 80% of the importance mass"): the smallest k such
    that the k largest scores sum to at least ``mass_fraction`` of the total.  Full sort, fp64 cumulative sum.
    Returns 0 for an all-zero vector."""
    s = np.sort(_f64(scores))[::-1]
    csum = np.cumsum(s)
    total = csum[-1] if len(csum) else 0.0            # the total is the last running sum: the full vector always suffices
    if not total > 0.0:
        return 0
    return min(len(s), int(np.searchsorted(csum, float(mass_fraction) * total, side="left")) + 1)


# ----------------------------------------------------------------------------
# block glue -- the paper gives only the recurrence; this is the standard Mamba-2 /
# pre-norm GQA block around it (parity unpinned by the paper)
# ----------------------------------------------------------------------------
def softplus(v):
    return np.logaddexp(0.0, v)


def silu(v):
    return v / (1.0 + np.exp(-v))


def rmsnorm(u, eps=1e-5):
    u = _f64(u)
    return u / np.sqrt((u * u).mean(axis=-1, keepdims=True) + eps)


def causal_conv1d_silu(v, w, bias):
    """out[t,c] = SiLU(bias[c] + sum_{j<W} w[c,j] * v[t-(W-1)+j, c]), zero left padding."""
    v, w, bias = _f64(v), _f64(w), _f64(bias)
    T, Cc = v.shape
    W = w.shape[1]
    out = np.tile(bias, (T, 1))
    for j in range(W):
        shift = W - 1 - j
        if shift < T:
            out[shift:] += w[:, j] * v[:T - shift]
    return silu(out)


def rope(v, positions, theta):
    """Rotary embedding, half-split pairing (i, i+d/2), angle = pos * theta^(-2i/d)."""
    v = _f64(v)
    T, Hh, d = v.shape
    half = d // 2
    inv = theta ** (-2.0 * np.arange(half) / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]     # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def attention_forward(q, k, v, scale, slab=512):
    """Causal GQA softmax attention, o_t = sum_{j<=t} softmax_j(q_t.k_j*scale) v_j.

    Rows are processed in slabs only to bound memory; each row's softmax is complete."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    o = np.zeros((T, Hq, d))
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        for s in range(0, T, slab):
            e = min(T, s + slab)
            logits = (q[s:e, h] @ k[:e, kv].T) * scale
            mask = np.arange(e)[None, :] > np.arange(s, e)[:, None]
            logits[mask] = -np.inf
            logits -= logits.max(axis=1, keepdims=True)
            w = np.exp(logits)
            w /= w.sum(axis=1, keepdims=True)
            o[s:e, h] = w @ v[:e, kv]
    return o


def attention_rows(q, k, v, scale, rows):
    """The same definition for a few query rows only: o_t for t in ``rows``, shape [len(rows), Hq, d].
    Used where the sequence is too long to evaluate every row on the CPU."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    o = np.zeros((len(rows), Hq, d))
    for i, t in enumerate(rows):
        for h in range(Hq):
            kv = h // (Hq // Hkv)
            logits = (k[:t + 1, kv] @ q[t, h]) * scale
            w = np.exp(logits - logits.max())
            o[i, h] = (w / w.sum()) @ v[:t + 1, kv]
    return o


def mamba2_block(u, prm, rnd=_identity):
    """One pre-norm Mamba-2 block.  prm: dict(H,p,n,G,W_in,conv_w,conv_b,dt_bias,A,W_out).

    Returns (layer output, dict of intermediates x,B,C,dt,y used by the score / tests).
    ``rnd`` is applied wherever the GPU path stores an activation (identity or bf16)."""
    H, p, n, G = prm["H"], prm["p"], prm["n"], prm["G"]
    d_inner = H * p
    u = _f64(u)
    T = u.shape[0]
    normed = rmsnorm(u)                        # not stored by the GPU path (the norm is fused into the projection)
    zxbcdt = rnd(normed @ _f64(prm["W_in"]))
    z = zxbcdt[:, :d_inner]
    xBC = zxbcdt[:, d_inner:2 * d_inner + 2 * G * n]
    dt_raw = zxbcdt[:, 2 * d_inner + 2 * G * n:]
    xBC = rnd(causal_conv1d_silu(xBC, prm["conv_w"], prm["conv_b"]))
    x = xBC[:, :d_inner].reshape(T, H, p)
    Bm = xBC[:, d_inner:d_inner + G * n].reshape(T, G, n)
    Cm = xBC[:, d_inner + G * n:].reshape(T, G, n)
    dt = softplus(dt_raw + _f64(prm["dt_bias"])[None, :])
    y, final_state = mamba2_recurrence(x, dt, prm["A"], Bm, Cm)
    y = rnd(y)
    gated = rnd(rmsnorm(y.reshape(T, d_inner) * silu(z)))
    out = rnd(u + gated @ _f64(prm["W_out"]))
    return out, dict(x=x, B=Bm, C=Cm, dt=dt, y=y, final_state=final_state)


def attn_block(u, positions, prm, rnd=_identity):
    """One pre-norm causal GQA attention block.  prm: dict(Hq,Hkv,d,theta,W_qkv,W_o)."""
    Hq, Hkv, d = prm["Hq"], prm["Hkv"], prm["d"]
    u = _f64(u)
    T = u.shape[0]
    normed = rmsnorm(u)                        # not stored by the GPU path (the norm is fused into the projection)
    qkv = rnd(normed @ _f64(prm["W_qkv"]))
    q = qkv[:, :Hq * d].reshape(T, Hq, d)
    k = qkv[:, Hq * d:(Hq + Hkv) * d].reshape(T, Hkv, d)
    v = qkv[:, (Hq + Hkv) * d:].reshape(T, Hkv, d)
    q = rnd(rope(q, positions, prm["theta"]))
    k = rnd(rope(k, positions, prm["theta"]))
    scale = 1.0 / np.sqrt(d)
    o = rnd(attention_forward(q, k, v, scale))
    out = rnd(u + o.reshape(T, Hq * d) @ _f64(prm["W_o"]))
    return out, dict(q=q, k=k, v=v, o=o, scale=scale)


def attn_block_projections(u, positions, prm, rnd=_identity):
    """The first half of attn_block: q, k (after the rotary embedding) and v of every row.  Returns dict(q, k, v, scale)."""
    Hq, Hkv, d = prm["Hq"], prm["Hkv"], prm["d"]
    u = _f64(u)
    T = u.shape[0]
    normed = rmsnorm(u)                        # not stored by the GPU path (the norm is fused into the projection)
    qkv = rnd(normed @ _f64(prm["W_qkv"]))
    q = qkv[:, :Hq * d].reshape(T, Hq, d)
    k = qkv[:, Hq * d:(Hq + Hkv) * d].reshape(T, Hkv, d)
    v = qkv[:, (Hq + Hkv) * d:].reshape(T, Hkv, d)
    q = rnd(rope(q, positions, prm["theta"]))
    k = rnd(rope(k, positions, prm["theta"]))
    return dict(q=q, k=k, v=v, scale=1.0 / np.sqrt(d))


def attn_block_rows(u, positions, prm, rows, rnd=_identity, mid=None):
    """attn_block for a sequence too long to evaluate every row on the CPU: q, k, v are computed for every row (or
    taken from ``mid`` = attn_block_projections of the same input), the attention output and the layer output only
    for ``rows``.  Returns (layer output rows [len(rows), D], mid)."""
    Hq, d = prm["Hq"], prm["d"]
    u = _f64(u)
    if mid is None:
        mid = attn_block_projections(u, positions, prm, rnd)
    rows = [int(r) for r in rows]
    o = rnd(attention_rows(mid["q"], mid["k"], mid["v"], mid["scale"], rows))
    out = rnd(u[rows] + o.reshape(len(rows), Hq * d) @ _f64(prm["W_o"]))
    return out, mid


def ffn_block(u, prm, rnd=_identity):
    """One pre-norm FFN block, u + W_down relu(W_up RMSNorm(u))^2.  prm: dict(D,F,W_up [D,F],W_down [F,D]).

    The paper names FFN (MLP) blocks as the third block type of its hybrid (appendix "Models") and says nothing
    about their inside; the squared-ReLU, ungated form is the one of the hybrid family it cites."""
    u = _f64(u)
    normed = rmsnorm(u)                        # not stored by the GPU path (the norm is fused into the projection)
    up = rnd(normed @ _f64(prm["W_up"]))
    act = rnd(np.maximum(up, 0.0) ** 2)
    return rnd(u + act @ _f64(prm["W_down"]))


def stack_prefill(hidden, n_text, layers, keep_counts, rnd=_identity, mamba_score="decoupled", attn_denominator="visual",
                  positions=None, idx_map=None, keep_inputs=False):
    """Token-reduced prefill of a layer stack (one sequence).

    hidden [T0,D] with the n_text text rows last; layers: list of ("M"|"A"|"F", prm);
    keep_counts[l] = visual tokens kept after layer l.  Layer l's mixer runs on the incoming
    tokens, its own score ranks the incoming visual tokens, and its OUTPUT is compacted when
    keep_counts[l] < n_cur.  Returns (hidden, positions, idx_map, trace) where trace lists per
    layer dict(n_in, scores or None, kept or None).  ``mamba_score``: "decoupled" (Eq. 2, the method) or
    "full_dynamic" (|w| of Eq. 1, the paper's scoring ablation); ``attn_denominator`` as in attn_importance.
    ``positions`` / ``idx_map``: original token ids of the incoming rows (default 0..T0-1), for continuing from a
    reduced context.  Every trace record also carries what a decoder would take over from the layer: the final
    recurrent state of a Mamba layer, the keys / values / positions of the rows leaving an attention layer; with
    ``keep_inputs`` it carries the layer's input (hidden, positions, idx_map) as well, for teacher-forced tests."""
    assert mamba_score in ("decoupled", "full_dynamic")
    h = _f64(hidden)
    T0 = h.shape[0]
    n_cur = T0 - n_text
    pos = np.arange(T0, dtype=np.int32) if positions is None else np.asarray(positions, dtype=np.int32).copy()
    idx = np.arange(T0, dtype=np.int32) if idx_map is None else np.asarray(idx_map, dtype=np.int32).copy()
    trace = []
    for (kind, prm), K in zip(layers, keep_counts):
        inputs = dict(hidden_in=h.copy(), positions_in=pos.copy(), idx_map_in=idx.copy()) if keep_inputs else {}
        if kind == "F":                                   # FFN layers transform the rows they get; they never score
            assert K == n_cur
            h = ffn_block(h, prm, rnd)
            trace.append(dict(n_in=n_cur, scores=None, kept=None, **inputs))
            continue
        if kind == "M":
            out, mid = mamba2_block(h, prm, rnd)
            if mamba_score == "full_dynamic":
                score = (lambda: mamba_importance_full_dynamic(mid["B"], mid["C"], mid["dt"], prm["A"], n_cur, n_text))
            else:
                score = (lambda: mamba_importance(mid["B"], mid["C"], mid["dt"], n_cur, n_text))
        else:
            out, mid = attn_block(h, pos, prm, rnd)
            score = (lambda: attn_importance(mid["q"], mid["k"], n_cur, n_text, mid["scale"], attn_denominator))
        rec = dict(n_in=n_cur, scores=None, kept=None, **inputs)
        rows_out = np.arange(n_cur + n_text)
        if K < n_cur:
            s = score()
            kept = topk_select(s, K)
            rows_out = np.concatenate([kept.astype(np.int64), np.arange(n_cur, n_cur + n_text)])
            out, pos, idx = compact(out, pos, idx, kept, n_text)
            rec.update(scores=s, kept=kept)
            n_cur = K
        if kind == "M":
            rec.update(final_state=mid["final_state"])
        else:
            rec.update(k=mid["k"][rows_out], v=mid["v"][rows_out], kv_positions=pos.copy())
        h = out
        trace.append(rec)
    return h, pos, idx, trace
