// extern "C" entry points of the hot path: argument validation and kernel selection.
#include "dispatch.cuh"

#include <stdlib.h>

#define STR_DTYPE_OK(dt) ((dt) == STR_F32 || (dt) == STR_BF16)

// Debug switch: STR_FORCE_SIMT=1 routes every call to the plain FFMA kernels (for A/B parity runs).
bool str_force_simt() {
    static int v = -1;
    if (v < 0) { const char *e = getenv("STR_FORCE_SIMT"); v = (e && e[0] == '1') ? 1 : 0; }
    return v == 1;
}

// ---------------------------------------------------------------- (1) Mamba-2 SSD scan
extern "C" size_t str_mamba2_prefill_workspace_size(const str_ssd_shape *s) {
    (void)s;
    return 0;
}

extern "C" int str_mamba2_prefill(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt,
                                  const float *A, const void *B, const void *C, const float *D,
                                  const float *init_state, void *y, float *final_state, void *workspace,
                                  size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_SSD, stream);
    (void)workspace;
    if (!ctx || !s || !x || !dt || !A || !B || !C || !y) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->T < 0 || s->H <= 0 || s->p <= 0 || s->n <= 0 || s->G <= 0 || s->H % s->G != 0 || s->Q < 0 ||
        !STR_DTYPE_OK(s->dtype))
        return STR_ERR_INVALID_ARG;
    if (workspace_bytes < str_mamba2_prefill_workspace_size(s)) return STR_ERR_WORKSPACE_TOO_SMALL;
    if (s->T == 0) return STR_OK;
    if (!str_force_simt() && ctx->encode_tiled && str_ssd_tc_supported(s, x, B, C, y, D, init_state))
        return ++ctx->tc_calls, str_ssd_tc(ctx, s, x, dt, A, B, C, y, final_state, (cudaStream_t)stream);
    if (!str_ssd_simt_supported(s)) return STR_ERR_UNSUPPORTED_SHAPE;
    return ++ctx->fallback_calls, str_ssd_simt(ctx, s, x, dt, A, B, C, D, init_state, y, final_state, (cudaStream_t)stream);
}

// ---------------------------------------------------------------- (2a) Mamba importance
extern "C" size_t str_mamba_importance_workspace_size(const str_ssm_score_shape *s, int n_vis, int n_text) {
    (void)s; (void)n_vis; (void)n_text;
    return 0;
}

extern "C" int str_mamba_importance(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text,
                                    const void *B, const void *C, const float *dt, float *scores_out,
                                    void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_MAMBA_SCORE, stream);
    (void)workspace; (void)workspace_bytes;
    if (!ctx || !s || !B || !C || !dt) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->H <= 0 || s->n <= 0 || s->G <= 0 || s->H % s->G != 0 || n_vis < 0 || n_text <= 0 ||
        n_vis + n_text != s->T || !STR_DTYPE_OK(s->dtype))
        return STR_ERR_INVALID_ARG;
    if (n_vis == 0) return STR_OK;
    if (!scores_out) return STR_ERR_INVALID_ARG;
    if (!str_force_simt() && ctx->encode_tiled && str_mamba_importance_tc_supported(s, n_vis, n_text, B, C))
        return ++ctx->tc_calls, str_mamba_importance_tc(ctx, s, n_vis, n_text, B, C, dt, scores_out, (cudaStream_t)stream);
    return ++ctx->fallback_calls, str_mamba_importance_simt(ctx, s, n_vis, n_text, B, C, dt, scores_out, (cudaStream_t)stream);
}

// ---------------------------------------------------------------- (2a') Mamba importance with the cumulative decay
// Workspace: chunk sums of dt A | U | V, where U, V are the decay weights in whichever layout is the larger.
static size_t dyn_uv_bytes(const str_ssm_score_shape *s, int n_vis, int n_text, bool split, size_t *u_bytes) {
    const size_t n_pad = (size_t)(n_text + 15) / 16 * 16;
    const size_t ub = split ? (size_t)s->Bz * n_vis * s->G * 64 * 2 : (size_t)s->Bz * n_vis * s->H * 4;
    const size_t vb = split ? (size_t)s->Bz * n_pad * s->G * 64 * 2 : (size_t)s->Bz * n_text * s->H * 4;
    if (u_bytes) *u_bytes = align_up(ub, 256);
    return align_up(ub, 256) + align_up(vb, 256);
}

extern "C" size_t str_mamba_importance_dynamic_workspace_size(const str_ssm_score_shape *s, int n_vis, int n_text) {
    if (!s || s->Bz <= 0 || s->H <= 0 || s->G <= 0 || n_vis <= 0 || n_text <= 0) return 0;
    const size_t a = dyn_uv_bytes(s, n_vis, n_text, false, nullptr), b = dyn_uv_bytes(s, n_vis, n_text, true, nullptr);
    return str_mamba_dyn_part_bytes(s, n_vis) + (a > b ? a : b);
}

extern "C" int str_mamba_importance_dynamic(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text,
                                            const void *B, const void *C, const float *dt, const float *A,
                                            float *scores_out, void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_MAMBA_SCORE, stream);
    if (!ctx || !s || !B || !C || !dt || !A) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->H <= 0 || s->n <= 0 || s->G <= 0 || s->H % s->G != 0 || n_vis < 0 || n_text <= 0 ||
        n_vis + n_text != s->T || !STR_DTYPE_OK(s->dtype))
        return STR_ERR_INVALID_ARG;
    if (n_vis == 0) return STR_OK;
    if (!scores_out || !workspace) return STR_ERR_INVALID_ARG;
    if (workspace_bytes < str_mamba_importance_dynamic_workspace_size(s, n_vis, n_text)) return STR_ERR_WORKSPACE_TOO_SMALL;
    const bool tc = !str_force_simt() && ctx->encode_tiled && str_mamba_dyn_importance_tc_supported(s, n_vis, n_text, B, C);
    const int n_pad = (n_text + 15) / 16 * 16;
    float *part = (float *)workspace;
    size_t u_bytes = 0;
    dyn_uv_bytes(s, n_vis, n_text, tc, &u_bytes);
    uint8_t *U = (uint8_t *)workspace + str_mamba_dyn_part_bytes(s, n_vis), *V = U + u_bytes;
    int rc = str_mamba_dyn_weights(ctx, s, n_vis, n_text, n_pad, dt, A, part, U, V, tc, (cudaStream_t)stream);
    if (rc != STR_OK) return rc;
    ++(tc ? ctx->tc_calls : ctx->fallback_calls);
    if (tc) return str_mamba_dyn_importance_tc(ctx, s, n_vis, n_text, B, C, U, V, scores_out, (cudaStream_t)stream);
    return str_mamba_dyn_importance_simt(ctx, s, n_vis, n_text, B, C, (const float *)U, (const float *)V, scores_out,
                                         (cudaStream_t)stream);
}

// ---------------------------------------------------------------- (2b) attention importance
extern "C" size_t str_attn_importance_workspace_size(const str_attn_score_shape *s, int n_vis, int n_text) {
    (void)n_vis;
    if (!s || s->Bz <= 0 || s->Hq <= 0 || n_text <= 0) return 0;
    // row maxima and sums per (sequence, head, key segment, text query), plus their merged form
    return align_up((size_t)2 * s->Bz * s->Hq * n_text * (STR_ATTN_SCORE_MAX_SEGMENTS + 1) * sizeof(float), 256);
}

extern "C" int str_attn_importance_ex(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                                      const void *q, const void *k, float softmax_scale, int denominator,
                                      float *scores_out, void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ATTN_SCORE, stream);
    if (!ctx || !s || !q || !k) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Hq % s->Hkv != 0 || s->d <= 0 || n_vis < 0 || n_text <= 0 ||
        n_vis + n_text != s->T || !STR_DTYPE_OK(s->dtype) ||
        (denominator != STR_ATTN_DENOM_VISUAL && denominator != STR_ATTN_DENOM_CAUSAL_ROW))
        return STR_ERR_INVALID_ARG;
    if (n_vis == 0) return STR_OK;
    if (!scores_out || !workspace) return STR_ERR_INVALID_ARG;
    if (workspace_bytes < str_attn_importance_workspace_size(s, n_vis, n_text)) return STR_ERR_WORKSPACE_TOO_SMALL;
    const bool causal_row = denominator == STR_ATTN_DENOM_CAUSAL_ROW;
    if (!str_force_simt() && ctx->encode_tiled && str_attn_importance_tc_supported(s, n_vis, n_text, q, k))
        return ++ctx->tc_calls, str_attn_importance_tc(ctx, s, n_vis, n_text, q, k, softmax_scale, scores_out, (float *)workspace,
                                                       causal_row, (cudaStream_t)stream);
    ++ctx->fallback_calls;
    float *row_max = (float *)workspace;
    float *row_sum = row_max + (size_t)s->Bz * s->Hq * n_text;
    return str_attn_importance_simt(ctx, s, n_vis, n_text, q, k, softmax_scale, scores_out, row_max, row_sum, causal_row,
                                    (cudaStream_t)stream);
}

extern "C" int str_attn_importance(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                                   const void *q, const void *k, float softmax_scale, float *scores_out,
                                   void *workspace, size_t workspace_bytes, void *stream) {
    return str_attn_importance_ex(ctx, s, n_vis, n_text, q, k, softmax_scale, STR_ATTN_DENOM_VISUAL, scores_out, workspace,
                                  workspace_bytes, stream);
}

// ---------------------------------------------------------------- glue: GEMM, attention forward
extern "C" size_t str_gemm_workspace_size(int, int, int, int) { return 0; }

int str_gemm_fused(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w, const void *residual, void *out,
                   const StrRowNorm &rn, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_GEMM, stream);
    if (!ctx || !a || !w || !out || M < 0 || N <= 0 || K <= 0 || !STR_DTYPE_OK(dtype)) return STR_ERR_INVALID_ARG;
    if (M == 0) return STR_OK;
    if (!str_force_simt() && ctx->encode_tiled && str_gemm_tc_supported(dtype, M, N, K, a, w, residual, out))
        return ++ctx->tc_calls, str_gemm_tc(ctx, M, N, K, a, w, residual, out, rn, StrConvEpilogue{}, (cudaStream_t)stream);
    return ++ctx->fallback_calls, str_gemm_simt(ctx, dtype, M, N, K, a, w, residual, out, rn, (cudaStream_t)stream);
}

extern "C" int str_gemm(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
                        const void *residual, void *out, void *workspace, size_t workspace_bytes, void *stream) {
    (void)workspace; (void)workspace_bytes;
    const StrRowNorm none = {nullptr, 0, 0.f, 0.f, nullptr};
    return str_gemm_fused(ctx, dtype, M, N, K, a, w, residual, out, none, stream);
}

extern "C" int str_mamba_in_proj_conv(str_ctx *ctx, int dtype, int Bz, int T, int D, int H, int p, int n, int G, int W,
                                      const void *u, const void *w_in, const float *conv_w, const float *conv_b,
                                      const float *dt_bias, void *zxbcdt, void *x_out, void *B_out, void *C_out,
                                      float *dt_out, void *stream) {
    if (!ctx || !u || !w_in || !conv_w || !conv_b || !dt_bias || !zxbcdt || !x_out || !B_out || !C_out || !dt_out || Bz <= 0 ||
        T <= 0 || D <= 0 || H <= 0 || p <= 0 || n <= 0 || G <= 0 || W <= 0 || !STR_DTYPE_OK(dtype))
        return STR_ERR_INVALID_ARG;
    if ((long long)Bz * T > 2147483647LL) return STR_ERR_UNSUPPORTED_SHAPE;
    const int rows = Bz * T, d_inner = H * p, gn = G * n, N = 2 * d_inner + 2 * gn + H;
    const StrRowNorm none = {nullptr, 0, 0.f, 0.f, nullptr};
    const StrConvEpilogue cv = {W == 4 ? T : 0, 0, d_inner, d_inner, gn, H, conv_w, conv_b, dt_bias, (__nv_bfloat16 *)x_out,
                                (__nv_bfloat16 *)B_out, (__nv_bfloat16 *)C_out, dt_out};
    if (!str_force_simt() && ctx->encode_tiled && str_gemm_conv_supported(dtype, rows, N, D, u, w_in, zxbcdt, cv)) {
        {
            StrProfScope prof_scope(ctx, STR_CAT_GEMM, stream);
            ++ctx->tc_calls;
            const int rc = str_gemm_tc(ctx, rows, N, D, u, w_in, nullptr, zxbcdt, none, cv, (cudaStream_t)stream);
            if (rc != STR_OK) return rc;
        }
        return str_mamba_conv_edge_rows(ctx, Bz, T, N, cv, zxbcdt, stream);
    }
    const int rc = str_gemm_fused(ctx, dtype, rows, N, D, u, w_in, nullptr, zxbcdt, none, stream);
    if (rc != STR_OK) return rc;
    return str_mamba_conv_split(ctx, dtype, Bz, T, H, p, n, G, W, zxbcdt, conv_w, conv_b, dt_bias, x_out, B_out, C_out, dt_out,
                                stream);
}

extern "C" size_t str_attn_prefill_workspace_size(const str_attn_shape *) { return 0; }

extern "C" int str_attn_prefill_rows(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q_rows,
                                     const int32_t *row_pos, const void *k, const void *v, float softmax_scale,
                                     void *o_rows, void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ATTN_FWD, stream);
    (void)workspace; (void)workspace_bytes;
    if (!ctx || !s || !q_rows || !k || !v || !o_rows) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->T <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Hq % s->Hkv != 0 || s->d <= 0 || n_rows < 0 ||
        !STR_DTYPE_OK(s->dtype) || (!row_pos && n_rows != s->T))
        return STR_ERR_INVALID_ARG;
    if (n_rows == 0) return STR_OK;
    if (!str_force_simt() && ctx->encode_tiled && str_attn_prefill_tc_supported(s, q_rows, k, v, o_rows))
        return ++ctx->tc_calls, str_attn_prefill_tc(ctx, s, n_rows, q_rows, row_pos, k, v, softmax_scale, o_rows, (cudaStream_t)stream);
    return ++ctx->fallback_calls, str_attn_prefill_simt(ctx, s, n_rows, q_rows, row_pos, k, v, softmax_scale, o_rows, (cudaStream_t)stream);
}

extern "C" int str_attn_prefill(str_ctx *ctx, const str_attn_shape *s, const void *q, const void *k, const void *v,
                                float softmax_scale, void *o, void *workspace, size_t workspace_bytes,
                                void *stream) {
    if (!s) return STR_ERR_INVALID_ARG;
    return str_attn_prefill_rows(ctx, s, s->T, q, nullptr, k, v, softmax_scale, o, workspace, workspace_bytes, stream);
}
