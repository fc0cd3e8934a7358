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
        return str_ssd_tc(ctx, s, x, dt, A, B, C, y, final_state, (cudaStream_t)stream);
    if (!str_ssd_simt_supported(s)) return STR_ERR_UNSUPPORTED_SHAPE;
    return str_ssd_simt(ctx, s, x, dt, A, B, C, D, init_state, y, final_state, (cudaStream_t)stream);
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
        return str_mamba_importance_tc(ctx, s, n_vis, n_text, B, C, dt, scores_out, (cudaStream_t)stream);
    return str_mamba_importance_simt(ctx, s, n_vis, n_text, B, C, dt, scores_out, (cudaStream_t)stream);
}

// ---------------------------------------------------------------- (2b) attention importance
extern "C" size_t str_attn_importance_workspace_size(const str_attn_score_shape *s, int n_vis, int n_text) {
    (void)n_vis;
    if (!s || s->Bz <= 0 || s->Hq <= 0 || n_text <= 0) return 0;
    // row maxima and sums per (sequence, head, key segment, text query), plus their merged form
    return align_up((size_t)2 * s->Bz * s->Hq * n_text * (STR_ATTN_SCORE_MAX_SEGMENTS + 1) * sizeof(float), 256);
}

extern "C" int str_attn_importance(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                                   const void *q, const void *k, float softmax_scale, float *scores_out,
                                   void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ATTN_SCORE, stream);
    if (!ctx || !s || !q || !k) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Hq % s->Hkv != 0 || s->d <= 0 || n_vis < 0 || n_text <= 0 ||
        n_vis + n_text != s->T || !STR_DTYPE_OK(s->dtype))
        return STR_ERR_INVALID_ARG;
    if (n_vis == 0) return STR_OK;
    if (!scores_out || !workspace) return STR_ERR_INVALID_ARG;
    if (workspace_bytes < str_attn_importance_workspace_size(s, n_vis, n_text)) return STR_ERR_WORKSPACE_TOO_SMALL;
    if (!str_force_simt() && ctx->encode_tiled && str_attn_importance_tc_supported(s, n_vis, n_text, q, k))
        return str_attn_importance_tc(ctx, s, n_vis, n_text, q, k, softmax_scale, scores_out, (float *)workspace,
                                      (cudaStream_t)stream);
    float *row_max = (float *)workspace;
    float *row_sum = row_max + (size_t)s->Bz * s->Hq * n_text;
    return str_attn_importance_simt(ctx, s, n_vis, n_text, q, k, softmax_scale, scores_out, row_max, row_sum,
                                    (cudaStream_t)stream);
}

// ---------------------------------------------------------------- glue: GEMM, attention forward
extern "C" size_t str_gemm_workspace_size(int, int, int, int) { return 0; }

extern "C" int str_gemm(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
                        const void *residual, void *out, void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_GEMM, stream);
    (void)workspace; (void)workspace_bytes;
    if (!ctx || !a || !w || !out || M < 0 || N <= 0 || K <= 0 || !STR_DTYPE_OK(dtype)) return STR_ERR_INVALID_ARG;
    if (M == 0) return STR_OK;
    if (!str_force_simt() && ctx->encode_tiled && str_gemm_tc_supported(dtype, M, N, K, a, w, residual, out))
        return str_gemm_tc(ctx, M, N, K, a, w, residual, out, (cudaStream_t)stream);
    return str_gemm_simt(ctx, dtype, M, N, K, a, w, residual, out, (cudaStream_t)stream);
}

extern "C" size_t str_attn_prefill_workspace_size(const str_attn_shape *) { return 0; }

extern "C" int str_attn_prefill(str_ctx *ctx, const str_attn_shape *s, const void *q, const void *k, const void *v,
                                float softmax_scale, void *o, void *workspace, size_t workspace_bytes,
                                void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ATTN_FWD, stream);
    (void)workspace; (void)workspace_bytes;
    if (!ctx || !s || !q || !k || !v || !o) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->T <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Hq % s->Hkv != 0 || s->d <= 0 ||
        !STR_DTYPE_OK(s->dtype))
        return STR_ERR_INVALID_ARG;
    if (!str_force_simt() && ctx->encode_tiled && str_attn_prefill_tc_supported(s, q, k, v, o))
        return str_attn_prefill_tc(ctx, s, q, k, v, softmax_scale, o, (cudaStream_t)stream);
    return str_attn_prefill_simt(ctx, s, q, k, v, softmax_scale, o, (cudaStream_t)stream);
}
