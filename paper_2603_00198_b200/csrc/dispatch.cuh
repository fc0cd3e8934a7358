// Internal entry points shared between translation units of libstr (not exported).
#pragma once
#include "common.cuh"

int str_mamba_importance_simt(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B,
                              const void *C, const float *dt, float *scores, cudaStream_t st);
int str_attn_importance_simt(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q,
                             const void *k, float scale, float *scores, float *row_max, float *row_sum,
                             bool causal_row, cudaStream_t st);
// Folds the text keys m' <= m into the first pass's row statistics (causal-row normalisation of the attention score).
int str_attn_text_keys_stats(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k,
                             float scale, bool log2_inv, float *st_max, float *st_sum, cudaStream_t st);
int str_ssd_simt(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt, const float *A,
                 const void *B, const void *C, const float *D, const float *init_state, void *y,
                 float *final_state, cudaStream_t st);
bool str_ssd_simt_supported(const str_ssd_shape *s);
// RMSNorm fused into a projection.  A pre-norm block computes RMSNorm(h) W^T; with unit norm weight the norm is a
// per-row scalar, so (h / rms) W^T = (h W^T) / rms: the GEMM runs on h itself and its epilogue scales row r by
// rsqrt(sum_j ss_in[r, j] * inv_dim + eps).  ss_in holds partial sums of squares of the stored values of row r of A,
// nt_in per row, written by the kernel that produced A: a GEMM given ss_out writes, per output row, one partial per
// STR_SS_BLOCK output columns ([M, ceil(N / STR_SS_BLOCK)] floats).  Partials are summed in index order, so the result
// does not depend on the order in which tiles finish.  All-null = plain GEMM.
#define STR_SS_BLOCK 256
struct StrRowNorm {
    const float *ss_in;
    int nt_in;
    float inv_dim, eps;
    float *ss_out;
};
static inline int str_ss_blocks(int N) { return (N + STR_SS_BLOCK - 1) / STR_SS_BLOCK; }
int str_gemm_fused(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w, const void *residual, void *out,
                   const StrRowNorm &rn, void *stream);
// Partial sums of squares of the rows of a [rows, D] matrix in the layout above (for a matrix no GEMM of this
// library produced: the stack's input).
int str_row_sumsq(str_ctx *ctx, int dtype, int rows, int D, const void *in, float *ss_out, void *stream);
int str_gemm_simt(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
                  const void *residual, void *out, const StrRowNorm &rn, cudaStream_t st);
// n_rows query rows per sequence; row_pos (device [Bz,n_rows], ascending) gives each row's index in the key sequence,
// nullptr = rows 0 .. n_rows-1 (then n_rows == s->T).
int str_attn_prefill_simt(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos,
                          const void *k, const void *v, float scale, void *o, cudaStream_t st);
bool str_gemm_tc_supported(int dtype, int M, int N, int K, const void *a, const void *w, const void *residual,
                           const void *out);
// The Mamba block's pre-scan step fused into the in-projection's epilogue.  The projection's output row is
// [z (zoff columns) | x (d_inner) | B (gn) | C (gn) | dt (H)].  With T != 0 the epilogue, instead of storing the
// x/B/C columns, applies the causal depthwise conv of width 4 along the rows (the three earlier rows of a warp's 32
// consecutive rows come from its neighbouring lanes), SiLU, and stores into the split x/B/C tensors; the dt columns
// become softplus(dt + dt_bias) in fp32.  Rows whose earlier rows belong to another warp (row % 32 < 3) are left to
// str_mamba_conv_edge_rows: for them and for the last three rows of every 32 the epilogue stores the projection
// itself, as the unfused GEMM would.  The arithmetic on every element is that of str_mamba_conv_split on the stored
// bf16 projection, so both routes give the same bits.  Column segments must start on multiples of 32.
struct StrConvEpilogue {
    int T;                       // rows per sequence; 0 = plain GEMM epilogue
    int row_base;                // index of the call's first row among the Bz * T rows (multiple of 32)
    int zoff, d_inner, gn, H;
    const float *conv_w, *conv_b, *dt_bias;
    __nv_bfloat16 *x_out, *B_out, *C_out;    // whole tensors (row 0 = first row of the first sequence)
    float *dt_out;
};
bool str_gemm_conv_supported(int dtype, int M, int N, int K, const void *a, const void *w, const void *out,
                             const StrConvEpilogue &cv);
int str_gemm_tc(str_ctx *ctx, int M, int N, int K, const void *a, const void *w, const void *residual, void *out,
                const StrRowNorm &rn, const StrConvEpilogue &cv, cudaStream_t st);
// Conv / SiLU / split of the rows the fused epilogue leaves out (row % 32 < 3), from the stored projection rows.
int str_mamba_conv_edge_rows(str_ctx *ctx, int Bz, int T, int ld, const StrConvEpilogue &cv, const void *zxbcdt, void *stream);
bool str_force_simt();
bool str_ssd_tc_supported(const str_ssd_shape *s, const void *x, const void *B, const void *C, const void *y,
                          const float *D, const float *init_state);
int str_ssd_tc(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt, const float *A, const void *B,
               const void *C, void *y, float *final_state, cudaStream_t st);
bool str_attn_prefill_tc_supported(const str_attn_shape *s, const void *q, const void *k, const void *v, const void *o);
int str_attn_prefill_tc(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos, const void *k,
                        const void *v, float scale, void *o, cudaStream_t st);
bool str_mamba_importance_tc_supported(const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C);
int str_mamba_importance_tc(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C,
                            const float *dt, float *scores, cudaStream_t st);
// "Full Mamba Dynamic" score: decay-weight pass (fp32 or bf16 high/low layout), then one of the two scoring kernels.
size_t str_mamba_dyn_part_bytes(const str_ssm_score_shape *s, int n_vis);
int str_mamba_dyn_weights(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, int n_pad, const float *dt,
                          const float *A, float *part, void *U, void *V, bool split, cudaStream_t st);
int str_mamba_dyn_importance_simt(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B,
                                  const void *C, const float *U, const float *V, float *scores, cudaStream_t st);
bool str_mamba_dyn_importance_tc_supported(const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C);
int str_mamba_dyn_importance_tc(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C,
                                const void *U, const void *V, float *scores, cudaStream_t st);
// Key segments the tensor-core attention score may split its first pass into (sizes the workspace).
#define STR_ATTN_SCORE_MAX_SEGMENTS 8
bool str_attn_importance_tc_supported(const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k);
int str_attn_importance_tc(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k,
                           float scale, float *scores, float *workspace, bool causal_row, cudaStream_t st);
// y rows gathered by `kept` (+ the text rows); z either gathered the same way or already compacted (z_compacted).
int str_gated_rmsnorm_gather(str_ctx *ctx, int dtype, int Bz, int T_in, int n_vis, int n_text, int k, int d_inner, int ld_z,
                             float eps, const void *y, const void *z, bool z_compacted, const int32_t *kept, void *out,
                             void *stream);
int str_mamba_conv_split_rows(str_ctx *ctx, int dtype, int Bz, int T, int H, int p, int n, int G, int W, bool has_z,
                              const void *zxbcdt, const float *conv_w, const float *conv_b, const float *dt_bias,
                              void *x_out, void *B_out, void *C_out, float *dt_out, void *stream);
