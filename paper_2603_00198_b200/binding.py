"""Thin ctypes binding over libstr.so: argument marshalling only.

Every function has the name of the C entry point it calls (see ``include/str.h``) and takes torch
CUDA tensors, which serve purely as device memory; all arithmetic runs in the library's kernels.
There is no fallback: if the library is missing or a call fails, an exception is raised.
"""
import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libstr.so")

STR_F32, STR_BF16 = 0, 1
STR_LAYER_MAMBA, STR_LAYER_ATTN, STR_LAYER_FFN = 0, 1, 2
STR_SCORE_DECOUPLED, STR_SCORE_FULL_DYNAMIC = 0, 1
c_int, c_float, c_size_t, c_void_p = ctypes.c_int, ctypes.c_float, ctypes.c_size_t, ctypes.c_void_p


class StrError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, lib().str_strerror(code).decode(), code))


class SsdShape(ctypes.Structure):
    _fields_ = [(k, c_int) for k in ("Bz", "T", "H", "p", "n", "G", "Q", "dtype")]


class SsmScoreShape(ctypes.Structure):
    _fields_ = [(k, c_int) for k in ("Bz", "T", "H", "n", "G", "dtype")]


class AttnScoreShape(ctypes.Structure):
    _fields_ = [(k, c_int) for k in ("Bz", "T", "Hq", "Hkv", "d", "dtype")]


class AttnShape(ctypes.Structure):
    _fields_ = [(k, c_int) for k in ("Bz", "T", "Hq", "Hkv", "d", "dtype")]


class Layer(ctypes.Structure):
    _fields_ = [("kind", c_int), ("w_in", c_void_p), ("w_out", c_void_p), ("conv_w", c_void_p),
                ("conv_b", c_void_p), ("dt_bias", c_void_p), ("A", c_void_p)]


class StackDesc(ctypes.Structure):
    _fields_ = ([(k, c_int) for k in ("Bz", "n_vis", "n_text", "D", "dtype", "H", "p", "n", "G", "Q",
                                      "conv_width", "Hq", "Hkv", "d")]
                + [("rope_theta", c_float), ("norm_eps", c_float), ("n_layers", c_int),
                   ("layers", ctypes.POINTER(Layer)), ("keep_counts", ctypes.POINTER(c_int)),
                   ("score_every_layer", c_int), ("mamba_score_kind", c_int), ("attn_score_denominator", c_int),
                   ("ffn_dim", c_int)])


class StackIO(ctypes.Structure):
    _fields_ = [("positions_in", c_void_p), ("idx_map_in", c_void_p), ("mamba_final_states", c_void_p),
                ("attn_k_out", c_void_p), ("attn_v_out", c_void_p), ("attn_pos_out", c_void_p)]


PROF_CATEGORIES = ["gemm", "ssd_scan", "mamba_score", "attn_score", "topk", "compact", "attn_fwd", "elementwise"]

EXPORTS = [
    "str_create", "str_destroy", "str_strerror", "str_check_status", "str_launch_count", "str_path_counts",
    "str_selftest_wait_timeout", "str_score_density", "str_schedule_keep_counts_layers",
    "str_profile_enable", "str_profile_collect",
    "str_mamba2_prefill_workspace_size", "str_mamba2_prefill",
    "str_mamba_importance_workspace_size", "str_mamba_importance",
    "str_mamba_importance_dynamic_workspace_size", "str_mamba_importance_dynamic",
    "str_attn_importance_workspace_size", "str_attn_importance", "str_attn_importance_ex", "str_attn_importance_static",
    "str_topk_select_workspace_size", "str_topk_select", "str_compact",
    "str_schedule_keep_counts", "str_sigmoid_schedule_bp",
    "str_gemm_workspace_size", "str_gemm", "str_rmsnorm", "str_relu_squared", "str_mamba_conv_split", "str_mamba_in_proj_conv",
    "str_gated_rmsnorm",
    "str_rope_split", "str_attn_prefill_workspace_size", "str_attn_prefill", "str_attn_prefill_rows",
    "str_stack_workspace_size", "str_stack_prefill", "str_stack_prefill_ex", "str_stack_host_workspace_size",
    "str_stack_prefill_host",
]

_LIB = None


def lib():
    """Load libstr.so once.  Raises if it has not been built (python -m paper_2603_00198_b200.build)."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libstr.so not found at %s; run `python -m paper_2603_00198_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        L.str_strerror.restype = ctypes.c_char_p
        L.str_launch_count.restype = ctypes.c_longlong
        L.str_launch_count.argtypes = [c_void_p]
        for name in EXPORTS:
            if name.endswith("_workspace_size"):
                getattr(L, name).restype = c_size_t
        _LIB = L
    return _LIB


def _dt(t):
    if t.dtype == torch.bfloat16:
        return STR_BF16
    if t.dtype == torch.float32:
        return STR_F32
    raise TypeError("unsupported dtype %s" % t.dtype)


def _p(t):
    if t is None:
        return c_void_p(None)
    if isinstance(t, int):
        return c_void_p(t)
    assert t.is_contiguous(), "tensors must be contiguous"
    return c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != 0:
        raise StrError(rc, where)


class Context:
    """Owns a str_ctx for one device plus a grow-only device workspace (a torch byte tensor)."""

    def __init__(self, device=0):
        if not torch.cuda.is_available():
            raise RuntimeError("libstr needs a CUDA device; there is no CPU path")
        self.device = device
        torch.cuda.set_device(device)
        self._h = c_void_p()
        _check(lib().str_create(c_int(device), ctypes.byref(self._h)), "str_create")
        self._ws = None

    def close(self):
        if self._h:
            lib().str_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    def workspace(self, nbytes):
        nbytes = max(int(nbytes), 256)
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda:%d" % self.device)
        return self._ws

    def check_status(self):
        _check(lib().str_check_status(self._h, _stream()), "str_check_status")

    def launch_count(self):
        return int(lib().str_launch_count(self._h))

    def path_counts(self):
        """(calls that ran a tensor-core kernel, calls that fell back to the fp32-FMA kernel)."""
        tc, fb = ctypes.c_longlong(), ctypes.c_longlong()
        _check(lib().str_path_counts(self._h, ctypes.byref(tc), ctypes.byref(fb)), "str_path_counts")
        return int(tc.value), int(fb.value)

    def selftest_wait_timeout(self, probe_limit=1000):
        _check(lib().str_selftest_wait_timeout(self._h, ctypes.c_uint(probe_limit), _stream()), "str_selftest_wait_timeout")

    def profile_enable(self, on=True):
        _check(lib().str_profile_enable(self._h, c_int(1 if on else 0)), "str_profile_enable")

    def profile_collect(self):
        """Returns {category: (milliseconds, calls)} accumulated since the last collect."""
        n = len(PROF_CATEGORIES)
        ms = (ctypes.c_double * n)()
        calls = (ctypes.c_longlong * n)()
        _check(lib().str_profile_collect(self._h, ms, calls, c_int(n)), "str_profile_collect")
        return {PROF_CATEGORIES[i]: (float(ms[i]), int(calls[i])) for i in range(n)}


def str_mamba2_prefill(ctx, x, dt, A, B, C, D=None, init_state=None, Q=0, want_final_state=False):
    Bz, T, H, p = x.shape
    G, n = B.shape[2], B.shape[3]
    s = SsdShape(Bz, T, H, p, n, G, Q, _dt(x))
    y = torch.empty_like(x)
    fs = torch.empty((Bz, H, p, n), dtype=torch.float32, device=x.device) if want_final_state else None
    nb = lib().str_mamba2_prefill_workspace_size(ctypes.byref(s))
    ws = ctx.workspace(nb)
    _check(lib().str_mamba2_prefill(ctx.handle, ctypes.byref(s), _p(x), _p(dt), _p(A), _p(B), _p(C), _p(D),
                                    _p(init_state), _p(y), _p(fs), _p(ws), c_size_t(ws.numel()), _stream()),
           "str_mamba2_prefill")
    return (y, fs) if want_final_state else y


def str_mamba_importance(ctx, B, C, dt, n_vis, n_text):
    Bz, T, G, n = B.shape
    H = dt.shape[2]
    s = SsmScoreShape(Bz, T, H, n, G, _dt(B))
    out = torch.empty((Bz, n_vis), dtype=torch.float32, device=B.device)
    nb = lib().str_mamba_importance_workspace_size(ctypes.byref(s), c_int(n_vis), c_int(n_text))
    ws = ctx.workspace(nb)
    _check(lib().str_mamba_importance(ctx.handle, ctypes.byref(s), c_int(n_vis), c_int(n_text), _p(B), _p(C), _p(dt),
                                      _p(out), _p(ws), c_size_t(ws.numel()), _stream()), "str_mamba_importance")
    return out


def str_mamba_importance_dynamic(ctx, B, C, dt, A, n_vis, n_text):
    Bz, T, G, n = B.shape
    H = dt.shape[2]
    s = SsmScoreShape(Bz, T, H, n, G, _dt(B))
    out = torch.empty((Bz, n_vis), dtype=torch.float32, device=B.device)
    nb = lib().str_mamba_importance_dynamic_workspace_size(ctypes.byref(s), c_int(n_vis), c_int(n_text))
    ws = ctx.workspace(nb)
    _check(lib().str_mamba_importance_dynamic(ctx.handle, ctypes.byref(s), c_int(n_vis), c_int(n_text), _p(B), _p(C),
                                              _p(dt), _p(A), _p(out), _p(ws), c_size_t(ws.numel()), _stream()),
           "str_mamba_importance_dynamic")
    return out


STR_ATTN_DENOM = {"visual": 0, "causal_row": 1}


def str_attn_importance(ctx, q, k, n_vis, n_text, softmax_scale, denominator="visual"):
    Bz, T, Hq, d = q.shape
    Hkv = k.shape[2]
    s = AttnScoreShape(Bz, T, Hq, Hkv, d, _dt(q))
    out = torch.empty((Bz, n_vis), dtype=torch.float32, device=q.device)
    nb = lib().str_attn_importance_workspace_size(ctypes.byref(s), c_int(n_vis), c_int(n_text))
    ws = ctx.workspace(nb)
    if denominator == "visual":
        _check(lib().str_attn_importance(ctx.handle, ctypes.byref(s), c_int(n_vis), c_int(n_text), _p(q), _p(k),
                                         c_float(softmax_scale), _p(out), _p(ws), c_size_t(ws.numel()), _stream()),
               "str_attn_importance")
    else:
        _check(lib().str_attn_importance_ex(ctx.handle, ctypes.byref(s), c_int(n_vis), c_int(n_text), _p(q), _p(k),
                                            c_float(softmax_scale), c_int(STR_ATTN_DENOM[denominator]), _p(out), _p(ws),
                                            c_size_t(ws.numel()), _stream()), "str_attn_importance_ex")
    return out


STR_ATTN_STATIC_MAX_ROWS = 65536


def str_attn_importance_static(ctx, q, k, n_vis, n_text, softmax_scale, out=None):
    """Allocation-free variant for callers that cannot allocate device memory: the scratch is a fixed
    array inside the library, so only inputs and the output buffer are passed (pass ``out`` to avoid
    even the output allocation this wrapper would otherwise make)."""
    Bz, T, Hq, d = q.shape
    Hkv = k.shape[2]
    s = AttnScoreShape(Bz, T, Hq, Hkv, d, _dt(q))
    if out is None:
        out = torch.empty((Bz, n_vis), dtype=torch.float32, device=q.device)
    _check(lib().str_attn_importance_static(ctx.handle, ctypes.byref(s), c_int(n_vis), c_int(n_text), _p(q), _p(k),
                                            c_float(softmax_scale), _p(out), _stream()), "str_attn_importance_static")
    return out


def str_topk_select(ctx, scores, k):
    Bz, n_vis = scores.shape
    out = torch.empty((Bz, k), dtype=torch.int32, device=scores.device)
    nb = lib().str_topk_select_workspace_size(c_int(Bz), c_int(n_vis), c_int(k))
    ws = ctx.workspace(nb)
    _check(lib().str_topk_select(ctx.handle, c_int(Bz), c_int(n_vis), c_int(k), _p(scores), _p(out), _p(ws),
                                 c_size_t(ws.numel()), _stream()), "str_topk_select")
    return out


def str_compact(ctx, hidden, positions, idx_map, kept_idx, n_text):
    Bz, T_in, D = hidden.shape
    k = kept_idx.shape[1]
    n_vis = T_in - n_text
    h_out = torch.empty((Bz, k + n_text, D), dtype=hidden.dtype, device=hidden.device)
    p_out = torch.empty((Bz, k + n_text), dtype=torch.int32, device=hidden.device) if positions is not None else None
    i_out = torch.empty((Bz, k + n_text), dtype=torch.int32, device=hidden.device) if idx_map is not None else None
    _check(lib().str_compact(ctx.handle, c_int(Bz), c_int(T_in), c_int(n_vis), c_int(n_text), c_int(k), c_int(D),
                             c_int(_dt(hidden)), _p(hidden), _p(positions), _p(idx_map), _p(kept_idx), _p(h_out),
                             _p(p_out), _p(i_out), _stream()), "str_compact")
    return h_out, p_out, i_out


def str_schedule_keep_counts(alpha_bp, n0, min_keep):
    L = len(alpha_bp)
    a = (c_int * L)(*[int(v) for v in alpha_bp])
    out = (c_int * L)()
    _check(lib().str_schedule_keep_counts(a, c_int(L), c_int(n0), c_int(min_keep), out), "str_schedule_keep_counts")
    return list(out)


LAYER_KIND = {"M": STR_LAYER_MAMBA, "A": STR_LAYER_ATTN, "F": STR_LAYER_FFN}


def str_schedule_keep_counts_layers(alpha_bp, pattern, n0, min_keep):
    """Keep counts for a stack whose layer kinds are given as a string of M / A / F: FFN layers never reduce."""
    L = len(alpha_bp)
    assert len(pattern) == L
    a = (c_int * L)(*[int(v) for v in alpha_bp])
    kinds = (c_int * L)(*[LAYER_KIND[c] for c in pattern])
    out = (c_int * L)()
    _check(lib().str_schedule_keep_counts_layers(a, kinds, c_int(L), c_int(n0), c_int(min_keep), out),
           "str_schedule_keep_counts_layers")
    return list(out)


def str_score_density(ctx, scores, mass_fraction):
    Bz, n_vis = scores.shape
    out = torch.empty((Bz,), dtype=torch.int32, device=scores.device)
    _check(lib().str_score_density(ctx.handle, c_int(Bz), c_int(n_vis), _p(scores), c_float(mass_fraction), _p(out), _stream()),
           "str_score_density")
    return out


def str_sigmoid_schedule_bp(L, k, x0, a_start, a_end):
    out = (c_int * L)()
    _check(lib().str_sigmoid_schedule_bp(c_int(L), ctypes.c_double(k), ctypes.c_double(x0), ctypes.c_double(a_start),
                                         ctypes.c_double(a_end), out), "str_sigmoid_schedule_bp")
    return list(out)


def str_gemm(ctx, a, w, residual=None):
    M, K = a.shape
    N = w.shape[0]
    assert w.shape[1] == K
    out = torch.empty((M, N), dtype=a.dtype, device=a.device)
    nb = lib().str_gemm_workspace_size(c_int(M), c_int(N), c_int(K), c_int(_dt(a)))
    ws = ctx.workspace(nb)
    _check(lib().str_gemm(ctx.handle, c_int(_dt(a)), c_int(M), c_int(N), c_int(K), _p(a), _p(w), _p(residual), _p(out),
                          _p(ws), c_size_t(ws.numel()), _stream()), "str_gemm")
    return out


def str_rmsnorm(ctx, x, eps=1e-5):
    rows, D = x.shape
    out = torch.empty_like(x)
    _check(lib().str_rmsnorm(ctx.handle, c_int(_dt(x)), c_int(rows), c_int(D), c_float(eps), _p(x), _p(out), _stream()),
           "str_rmsnorm")
    return out


def str_relu_squared(ctx, x, inplace=False):
    out = x if inplace else torch.empty_like(x)
    _check(lib().str_relu_squared(ctx.handle, c_int(_dt(x)), c_size_t(x.numel()), _p(x), _p(out), _stream()),
           "str_relu_squared")
    return out


def str_mamba_conv_split(ctx, zxbcdt, conv_w, conv_b, dt_bias, Bz, T, H, p, n, G):
    W = conv_w.shape[1]
    dev, dtp = zxbcdt.device, zxbcdt.dtype
    x = torch.empty((Bz, T, H, p), dtype=dtp, device=dev)
    Bm = torch.empty((Bz, T, G, n), dtype=dtp, device=dev)
    Cm = torch.empty((Bz, T, G, n), dtype=dtp, device=dev)
    dt = torch.empty((Bz, T, H), dtype=torch.float32, device=dev)
    _check(lib().str_mamba_conv_split(ctx.handle, c_int(_dt(zxbcdt)), c_int(Bz), c_int(T), c_int(H), c_int(p), c_int(n),
                                      c_int(G), c_int(W), _p(zxbcdt), _p(conv_w), _p(conv_b), _p(dt_bias), _p(x),
                                      _p(Bm), _p(Cm), _p(dt), _stream()), "str_mamba_conv_split")
    return x, Bm, Cm, dt


def str_mamba_in_proj_conv(ctx, u, w_in, conv_w, conv_b, dt_bias, Bz, T, H, p, n, G):
    """In-projection of the rows u [Bz*T, D] and the pre-scan step in one call; returns (zxbcdt, x, B, C, dt), of
    zxbcdt only the first H*p columns (the gate z) are meaningful."""
    W = conv_w.shape[1]
    dev, dtp = u.device, u.dtype
    D = u.shape[1]
    N = 2 * H * p + 2 * G * n + H
    assert u.shape[0] == Bz * T and tuple(w_in.shape) == (N, D)
    zx = torch.empty((Bz * T, N), dtype=dtp, device=dev)
    x = torch.empty((Bz, T, H, p), dtype=dtp, device=dev)
    Bm = torch.empty((Bz, T, G, n), dtype=dtp, device=dev)
    Cm = torch.empty((Bz, T, G, n), dtype=dtp, device=dev)
    dt = torch.empty((Bz, T, H), dtype=torch.float32, device=dev)
    _check(lib().str_mamba_in_proj_conv(ctx.handle, c_int(_dt(u)), c_int(Bz), c_int(T), c_int(D), c_int(H), c_int(p), c_int(n),
                                        c_int(G), c_int(W), _p(u), _p(w_in), _p(conv_w), _p(conv_b), _p(dt_bias), _p(zx), _p(x),
                                        _p(Bm), _p(Cm), _p(dt), _stream()), "str_mamba_in_proj_conv")
    return zx, x, Bm, Cm, dt


def str_gated_rmsnorm(ctx, y, zxbcdt, d_inner, eps=1e-5):
    rows = y.shape[0]
    out = torch.empty_like(y)
    _check(lib().str_gated_rmsnorm(ctx.handle, c_int(_dt(y)), c_int(rows), c_int(d_inner), c_int(zxbcdt.shape[1]),
                                   c_float(eps), _p(y), _p(zxbcdt), _p(out), _stream()), "str_gated_rmsnorm")
    return out


def str_rope_split(ctx, qkv, positions, Bz, T, Hq, Hkv, d, theta):
    dev, dtp = qkv.device, qkv.dtype
    q = torch.empty((Bz, T, Hq, d), dtype=dtp, device=dev)
    k = torch.empty((Bz, T, Hkv, d), dtype=dtp, device=dev)
    v = torch.empty((Bz, T, Hkv, d), dtype=dtp, device=dev)
    _check(lib().str_rope_split(ctx.handle, c_int(_dt(qkv)), c_int(Bz), c_int(T), c_int(Hq), c_int(Hkv), c_int(d),
                                c_float(theta), _p(positions), _p(qkv), _p(q), _p(k), _p(v), _stream()),
           "str_rope_split")
    return q, k, v


def str_attn_prefill(ctx, q, k, v, softmax_scale):
    Bz, T, Hq, d = q.shape
    Hkv = k.shape[2]
    s = AttnShape(Bz, T, Hq, Hkv, d, _dt(q))
    o = torch.empty_like(q)
    nb = lib().str_attn_prefill_workspace_size(ctypes.byref(s))
    ws = ctx.workspace(nb)
    _check(lib().str_attn_prefill(ctx.handle, ctypes.byref(s), _p(q), _p(k), _p(v), c_float(softmax_scale), _p(o),
                                  _p(ws), c_size_t(ws.numel()), _stream()), "str_attn_prefill")
    return o


def str_attn_prefill_rows(ctx, q_rows, row_pos, k, v, softmax_scale):
    """Attention outputs of a gathered subset of query rows: q_rows [Bz,n_rows,Hq,d], row_pos [Bz,n_rows] int32."""
    Bz, n_rows, Hq, d = q_rows.shape
    T, Hkv = k.shape[1], k.shape[2]
    s = AttnShape(Bz, T, Hq, Hkv, d, _dt(q_rows))
    o = torch.empty_like(q_rows)
    ws = ctx.workspace(256)
    _check(lib().str_attn_prefill_rows(ctx.handle, ctypes.byref(s), c_int(n_rows), _p(q_rows), _p(row_pos), _p(k), _p(v),
                                       c_float(softmax_scale), _p(o), _p(ws), c_size_t(ws.numel()), _stream()),
           "str_attn_prefill_rows")
    return o


class Stack:
    """Device-resident parameters of a layer stack plus the str_stack_desc that describes it.

    ``layers`` is the list produced by ``inputs.stack_params`` (host numpy, weights stored
    [in_features, out_features]); they are uploaded once, transposed to the library's
    [out_features, in_features] layout."""

    def __init__(self, ctx, layers, dtype, Bz, n_vis, n_text, keep_counts, Q=0, score_every_layer=False,
                 rope_theta=1.0e6, norm_eps=1e-5, mamba_score="decoupled", attn_denominator="visual"):
        self.ctx = ctx
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        dev = "cuda:%d" % ctx.device
        self._keep = []          # keeps device tensors alive
        arr = (Layer * len(layers))()
        m_shape = a_shape = None
        D = None
        ffn_dim = 0
        for i, (kind, prm) in enumerate(layers):
            def up(a, t=tdt):
                ten = torch.from_numpy(a).to(dev).to(t).contiguous()
                self._keep.append(ten)
                return ten.data_ptr()
            D = prm["D"]
            if kind == "M":
                m_shape = prm
                arr[i] = Layer(STR_LAYER_MAMBA, up(prm["W_in"].T.copy()), up(prm["W_out"].T.copy()),
                               up(prm["conv_w"], torch.float32), up(prm["conv_b"], torch.float32),
                               up(prm["dt_bias"], torch.float32), up(prm["A"], torch.float32))
            elif kind == "F":
                ffn_dim = prm["F"]
                arr[i] = Layer(STR_LAYER_FFN, up(prm["W_up"].T.copy()), up(prm["W_down"].T.copy()), None, None, None, None)
            else:
                a_shape = prm
                rope_theta = prm["theta"]
                arr[i] = Layer(STR_LAYER_ATTN, up(prm["W_qkv"].T.copy()), up(prm["W_o"].T.copy()), None, None, None,
                               None)
        self._layers = arr
        self._kc = (c_int * len(layers))(*[int(k) for k in keep_counts])
        ms = m_shape or dict(H=0, p=0, n=0, G=0)
        as_ = a_shape or dict(Hq=0, Hkv=0, d=0)
        self.desc = StackDesc(Bz, n_vis, n_text, D, STR_BF16 if dtype == "bf16" else STR_F32,
                              ms["H"], ms["p"], ms["n"], ms["G"], Q, 4 if m_shape else 0,
                              as_["Hq"], as_["Hkv"], as_["d"], rope_theta, norm_eps, len(layers),
                              ctypes.cast(arr, ctypes.POINTER(Layer)), ctypes.cast(self._kc, ctypes.POINTER(c_int)),
                              1 if score_every_layer else 0,
                              {"decoupled": STR_SCORE_DECOUPLED, "full_dynamic": STR_SCORE_FULL_DYNAMIC}[mamba_score],
                              STR_ATTN_DENOM[attn_denominator], ffn_dim)
        self.tdt, self.dev = tdt, dev
        self.Bz, self.n_vis, self.n_text, self.D = Bz, n_vis, n_text, D
        self.keep_counts = [int(k) for k in keep_counts]
        self.K_last = self.keep_counts[-1]
        n_cur, self.trace_layout = n_vis, []
        for l, K in enumerate(self.keep_counts):
            if K < n_cur:
                self.trace_layout.append((l, n_cur, K))
                n_cur = K
        self.ws_bytes = lib().str_stack_workspace_size(ctypes.byref(self.desc))
        self.host_ws_bytes = lib().str_stack_host_workspace_size(ctypes.byref(self.desc))
        if self.ws_bytes == 0:
            raise StrError(-1, "str_stack_workspace_size")


def str_stack_prefill(stack, hidden_in, want_trace=False):
    """Runs the stack on device-resident hidden states [Bz, n_vis+n_text, D]."""
    ctx = stack.ctx
    T_out = stack.K_last + stack.n_text
    out = torch.empty((stack.Bz, T_out, stack.D), dtype=stack.tdt, device=stack.dev)
    pos = torch.empty((stack.Bz, T_out), dtype=torch.int32, device=stack.dev)
    idx = torch.empty((stack.Bz, T_out), dtype=torch.int32, device=stack.dev)
    kept_tr = score_tr = None
    if want_trace and stack.trace_layout:
        kept_tr = torch.empty(sum(stack.Bz * K for _, _, K in stack.trace_layout), dtype=torch.int32, device=stack.dev)
        score_tr = torch.empty(sum(stack.Bz * n for _, n, _ in stack.trace_layout), dtype=torch.float32, device=stack.dev)
    ws = ctx.workspace(stack.ws_bytes)
    _check(lib().str_stack_prefill(ctx.handle, ctypes.byref(stack.desc), _p(hidden_in), _p(out), _p(pos), _p(idx),
                                   _p(kept_tr), _p(score_tr), _p(ws), c_size_t(ws.numel()), _stream()),
           "str_stack_prefill")
    if not want_trace:
        return out, pos, idx
    trace, ko, so = [], 0, 0
    for l, n_in, K in stack.trace_layout:
        trace.append(dict(layer=l, n_in=n_in, kept=kept_tr[ko:ko + stack.Bz * K].view(stack.Bz, K),
                          scores=score_tr[so:so + stack.Bz * n_in].view(stack.Bz, n_in)))
        ko += stack.Bz * K
        so += stack.Bz * n_in
    return out, pos, idx, trace


def str_stack_prefill_ex(stack, hidden_in, positions_in=None, idx_map_in=None, want_handoff=False, want_trace=False):
    """str_stack_prefill with the optional inputs (original token ids of the incoming rows) and, with
    ``want_handoff``, the decoder hand-off outputs: the final state of every Mamba layer and the keys, values and
    positions of the rows leaving every attention layer.  Returns a dict (``trace`` as in str_stack_prefill)."""
    ctx = stack.ctx
    T_out = stack.K_last + stack.n_text
    out = torch.empty((stack.Bz, T_out, stack.D), dtype=stack.tdt, device=stack.dev)
    pos = torch.empty((stack.Bz, T_out), dtype=torch.int32, device=stack.dev)
    idx = torch.empty((stack.Bz, T_out), dtype=torch.int32, device=stack.dev)
    d = stack.desc
    kinds = [stack._layers[i].kind for i in range(d.n_layers)]
    states, ks, vs, kvpos = [], [], [], []
    fs_all = k_all = v_all = p_all = None
    if want_handoff:
        n_m = sum(1 for k in kinds if k == STR_LAYER_MAMBA)
        rows_a = [stack.Bz * (stack.keep_counts[l] + stack.n_text) for l, k in enumerate(kinds) if k == STR_LAYER_ATTN]
        if n_m:
            fs_all = torch.empty((n_m, stack.Bz, d.H, d.p, d.n), dtype=torch.float32, device=stack.dev)
        if rows_a:
            k_all = torch.empty((sum(rows_a), d.Hkv, d.d), dtype=stack.tdt, device=stack.dev)
            v_all = torch.empty_like(k_all)
            p_all = torch.empty((sum(rows_a),), dtype=torch.int32, device=stack.dev)
    io = StackIO(_p(positions_in), _p(idx_map_in), _p(fs_all), _p(k_all), _p(v_all), _p(p_all))
    kept_tr = score_tr = None
    if want_trace and stack.trace_layout:
        kept_tr = torch.empty(sum(stack.Bz * K for _, _, K in stack.trace_layout), dtype=torch.int32, device=stack.dev)
        score_tr = torch.empty(sum(stack.Bz * n for _, n, _ in stack.trace_layout), dtype=torch.float32, device=stack.dev)
    ws = ctx.workspace(stack.ws_bytes)
    _check(lib().str_stack_prefill_ex(ctx.handle, ctypes.byref(stack.desc), ctypes.byref(io), _p(hidden_in), _p(out), _p(pos),
                                      _p(idx), _p(kept_tr), _p(score_tr), _p(ws), c_size_t(ws.numel()), _stream()),
           "str_stack_prefill_ex")
    res = dict(hidden=out, positions=pos, idx_map=idx)
    if want_trace:
        trace, ko, so = [], 0, 0
        for l, n_in, K in stack.trace_layout:
            trace.append(dict(layer=l, n_in=n_in, kept=kept_tr[ko:ko + stack.Bz * K].view(stack.Bz, K),
                              scores=score_tr[so:so + stack.Bz * n_in].view(stack.Bz, n_in)))
            ko += stack.Bz * K
            so += stack.Bz * n_in
        res["trace"] = trace
    if want_handoff:
        mi, ro = 0, 0
        for l, k in enumerate(kinds):
            if k == STR_LAYER_MAMBA:
                states.append((l, fs_all[mi]))
                mi += 1
            elif k == STR_LAYER_ATTN:
                n = stack.Bz * (stack.keep_counts[l] + stack.n_text)
                shp = (stack.Bz, stack.keep_counts[l] + stack.n_text)
                ks.append((l, k_all[ro:ro + n].view(*shp, d.Hkv, d.d)))
                vs.append((l, v_all[ro:ro + n].view(*shp, d.Hkv, d.d)))
                kvpos.append((l, p_all[ro:ro + n].view(*shp)))
                ro += n
        res.update(mamba_final_states=states, attn_k=ks, attn_v=vs, attn_pos=kvpos)
    return res


def str_stack_prefill_host(stack, hidden_in_host, hidden_out_host, idx_out_host):
    """Host-buffer entry point: pinned host tensors in and out; copies are inside the call."""
    ctx = stack.ctx
    ws = ctx.workspace(stack.host_ws_bytes)
    _check(lib().str_stack_prefill_host(ctx.handle, ctypes.byref(stack.desc), c_void_p(hidden_in_host.data_ptr()),
                                        c_void_p(hidden_out_host.data_ptr()), c_void_p(idx_out_host.data_ptr()),
                                        _p(ws), c_size_t(ws.numel()), _stream()), "str_stack_prefill_host")
