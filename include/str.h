/*
 * libstr -- token-reduced prefill of a hybrid Mamba-2 / attention layer stack, B200 (sm_100a).
 *
 * C ABI.  Conventions shared by every call:
 *   - returns int: STR_OK (0) or a negative STR_ERR_* code; str_strerror() gives text.
 *   - pointers named *_dev / documented "device" are DEVICE pointers owned by the caller; all
 *     tensors are row-major and contiguous in the layout stated.  "host" pointers are host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work: they never allocate, free or synchronise, unless stated otherwise.
 *   - scratch memory comes from a caller-provided device workspace whose size the matching
 *     *_workspace_size() query returns (bytes; 256-byte aligned base expected).
 *   - outputs are fully overwritten; inputs are never modified; in and out must not alias.
 *   - dtype is STR_F32 (everything fp32) or STR_BF16 (bf16 storage, fp32 accumulation).
 *   - bounded device-side waits: a kernel that gives up waiting records STR_ERR_TIMEOUT in the
 *     context's device status word and returns; str_check_status() reads it back.
 * Token order inside a sequence follows the paper's setting (Section 3.1): the n_vis visual
 * tokens come first, the n_text text (query) tokens last; text tokens are never dropped.
 */
#ifndef STR_H_
#define STR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    STR_OK = 0,
    STR_ERR_INVALID_ARG = -1,
    STR_ERR_UNSUPPORTED_SHAPE = -2,
    STR_ERR_WORKSPACE_TOO_SMALL = -3,
    STR_ERR_CUDA = -4,
    STR_ERR_TIMEOUT = -5
};

enum { STR_F32 = 0, STR_BF16 = 1 };

typedef struct str_ctx str_ctx;

/* Context: device id, SM count, tensor-map encoder, device status word.  str_create allocates
 * a few bytes of device memory and may synchronise; str_destroy frees them.  str_create fails with
 * STR_ERR_CUDA when the driver offers no tensor-map encoder: without it no tensor-core kernel can run
 * and every call would silently take the much slower fp32-FMA kernels. */
int str_create(int device, str_ctx **out);
int str_destroy(str_ctx *ctx);
const char *str_strerror(int code);
/* Synchronises `stream`, returns the device status word (STR_OK or the first recorded error)
 * and clears it.  The only hot-path call that synchronises. */
int str_check_status(str_ctx *ctx, void *stream);

/* ------------------------------------------------------------------------------------------
 * (1) Mamba-2 selective state-space scan.  Section 3.1 "State-Space (Mamba) Layers" and the
 * appendix "State-Space Recurrence":  S_t = Abar_t S_{t-1} + x_t (Delta_t b_t)^T,  y_t = S_t c_t,
 * Abar_t = exp(Delta_t * A_h) with the stored A_h < 0 (the paper writes exp(-Delta A), A > 0).
 * Evaluated in chunked form (in-chunk cumulative log-decay, intra-chunk (C B^T o decay) X,
 * chunk states, inter-chunk carry); the result equals the sequential recurrence up to fp32
 * rounding and does not depend on the chunk length.
 *   x   device [Bz,T,H,p] dtype        dt  device [Bz,T,H] fp32 (> 0, after softplus)
 *   A   device [H] fp32 (< 0)          B,C device [Bz,T,G,n] dtype (head h uses group h/(H/G))
 *   D   device [H] fp32 or NULL (y_t += D_h x_t)     init_state device [Bz,H,p,n] fp32 or NULL
 *   y   device [Bz,T,H,p] dtype        final_state device [Bz,H,p,n] fp32 or NULL
 * Q is a chunk-length hint (0 = library default); T need not be a multiple of it.
 * Errors: INVALID_ARG (null pointer, non-positive size, H % G != 0), UNSUPPORTED_SHAPE
 * (p or n beyond what the kernels tile), WORKSPACE_TOO_SMALL. */
typedef struct {
    int Bz, T, H, p, n, G, Q, dtype;
} str_ssd_shape;
size_t str_mamba2_prefill_workspace_size(const str_ssd_shape *s);
int str_mamba2_prefill(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt,
                       const float *A, const void *B, const void *C, const float *D,
                       const float *init_state, void *y, float *final_state, void *workspace,
                       size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * (2a) Mamba importance, Eq. 2 (Decoupled Content Alignment, decay excluded):
 *   s_i = 1/(M G) sum_{m,g} | (Deltabar_i^(g) b_i^(g))^T c_m^(g) |,
 * Deltabar_i^(g) = mean of dt[i,h] over the heads of group g; i over the first n_vis rows,
 * m over the last n_text rows of the same B, C, dt buffers the scan reads.
 *   scores_out device [Bz,n_vis] fp32.   n_vis + n_text must equal T. */
typedef struct {
    int Bz, T, H, n, G, dtype;
} str_ssm_score_shape;
size_t str_mamba_importance_workspace_size(const str_ssm_score_shape *s, int n_vis, int n_text);
int str_mamba_importance(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text,
                         const void *B, const void *C, const float *dt, float *scores_out,
                         void *workspace, size_t workspace_bytes, void *stream);

/* (2a', score variant)  "Full Mamba Dynamic", Section 3.1 (the paragraph on why it fails) and Eq. 1: the
 * magnitude of the exact weight w_{t,i} with which visual token i enters the output at text position t,
 *   s_i = 1/(M H) sum_{m,h} | (prod_{u=i+1..t_m} Abar_u^(h)) (dt[i,h] b_i^(g(h)))^T c_{t_m}^(g(h)) |,
 * Abar_u^(h) = exp(dt[u,h] A[h]), t_m = n_vis + m.  The paper uses it as the ablation against Eq. 2 (its
 * scoring-ablation table); the mean over text positions and heads is this library's reading.
 *   B, C device [Bz,T,G,n] dtype; dt device [Bz,T,H] fp32 (post-softplus); A device [H] fp32 (< 0);
 *   scores_out device [Bz,n_vis] fp32 (tokens far from the text underflow to 0: that is the score's nature).
 * Workspace (caller-owned, size from the query) holds the per-token decay weights.  Errors as (2a). */
size_t str_mamba_importance_dynamic_workspace_size(const str_ssm_score_shape *s, int n_vis, int n_text);
int str_mamba_importance_dynamic(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text,
                                 const void *B, const void *C, const float *dt, const float *A,
                                 float *scores_out, void *workspace, size_t workspace_bytes, void *stream);

/* (2b) Attention importance, Section 3.1 "Attention Layers":
 *   s_i = 1/(M Hq) sum_{m,h} softmax_i( q_m^(h) . k_i^(kv(h)) * softmax_scale ),
 * softmax over the n_vis visual keys, m over the last n_text query rows, kv(h) = h/(Hq/Hkv).
 *   q device [Bz,T,Hq,d] dtype (post-RoPE), k device [Bz,T,Hkv,d] dtype (post-RoPE),
 *   scores_out device [Bz,n_vis] fp32.  Workspace holds the per-(head, query) row maxima and
 *   sums of the first pass. */
typedef struct {
    int Bz, T, Hq, Hkv, d, dtype;
} str_attn_score_shape;
/* Normaliser of the attention score.  VISUAL: the paper's formula, softmax over the visual keys (scores sum to 1).
 * CAUSAL_ROW: the denominator of the model's own causal attention row, which also holds the text keys m' <= m;
 * the score is then the probability mass the text queries really put on each visual token (sums to < 1). */
enum { STR_ATTN_DENOM_VISUAL = 0, STR_ATTN_DENOM_CAUSAL_ROW = 1 };
size_t str_attn_importance_workspace_size(const str_attn_score_shape *s, int n_vis, int n_text);
int str_attn_importance(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                        const void *q, const void *k, float softmax_scale, float *scores_out,
                        void *workspace, size_t workspace_bytes, void *stream);
/* Same with the normaliser chosen by `denominator` (STR_ATTN_DENOM_*); str_attn_importance is the VISUAL case.
 * Same workspace size. */
int str_attn_importance_ex(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                           const void *q, const void *k, float softmax_scale, int denominator,
                           float *scores_out, void *workspace, size_t workspace_bytes, void *stream);

/* (2b, allocation-free variant)  The paper has no counterpart for this call; it exists for callers
 * that cannot allocate device memory (a plug-in inside a host with a fixed memory pool, a real-time
 * loop that must stay off the allocator, code that is handed raw pointers and owns no allocator).
 * Same inputs and outputs as str_attn_importance, but the per-(sequence, head, query) row maxima and
 * sums live in a fixed array inside the library image, so no workspace is passed and the call itself
 * allocates nothing.  It always runs the plain fp32-FMA kernels (never the tensor-core path), so for
 * bf16 inputs with head dimension 128 its scores agree with str_attn_importance to the score tolerance
 * (1e-3 relative), not bit for bit, and it is slower at large shapes.
 *   Limit: Bz * Hq * n_text <= STR_ATTN_STATIC_MAX_ROWS, else STR_ERR_WORKSPACE_TOO_SMALL is
 *   returned and nothing is launched.  The array (2 * STR_ATTN_STATIC_MAX_ROWS floats = 512 KiB) is
 *   resident on every GPU that loads the library until the process exits; it becomes resident when
 *   the driver loads the library's device code, which with lazy module loading may be during the
 *   first call.
 *   The first call on a device looks up the array's device address (one runtime query, no
 *   allocation); make that first call before starting any stream capture.
 *   All calls share the array and it keeps the previous call's contents; each call overwrites the
 *   part it uses before reading it, so nothing needs clearing, but two calls whose kernels overlap
 *   on the GPU (different streams, no ordering between them) race on it: serialise them. */
#define STR_ATTN_STATIC_MAX_ROWS 65536
int str_attn_importance_static(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                               const void *q, const void *k, float softmax_scale, float *scores_out,
                               void *stream);

/* ------------------------------------------------------------------------------------------
 * (3) Top-K selection preserving temporal order (Section 3.1 "Token Selection"): the indices of
 * the k largest scores of each row, written in ascending index order.  Among equal scores the
 * lower index is kept.  Radix select on the order-preserving integer image of fp32.
 *   scores device [Bz,n_vis] fp32 (any finite values; NaN unsupported),
 *   kept_idx_out device [Bz,k] int32.  k == n_vis gives 0..n_vis-1; k == 0 writes nothing;
 *   k > n_vis or k < 0 -> INVALID_ARG.
 * Workspace: none for rows of up to 131072 scores.  Longer rows are split over many CTAs that meet in the
 * workspace (256-byte aligned, size from the query); without it they are still selected correctly, by one
 * CTA per row that re-reads the row on every pass. */
size_t str_topk_select_workspace_size(int Bz, int n_vis, int k);
int str_topk_select(str_ctx *ctx, int Bz, int n_vis, int k, const float *scores,
                    int32_t *kept_idx_out, void *workspace, size_t workspace_bytes, void *stream);

/* (4) Compaction ("retain the top-K tokens", Section 3.1): per sequence, output row j < k is
 * input row kept_idx[j]; output rows k .. k+n_text-1 are the text rows n_vis .. n_vis+n_text-1.
 * The same gather is applied to hidden states, positions and the index map (which therefore
 * composes back to original token ids over several reductions).  Bit-exact copy.
 *   hidden device [Bz,T_in,D] dtype, positions/idx_map device [Bz,T_in] int32,
 *   kept_idx device [Bz,k] int32 (ascending, each in [0,n_vis)),
 *   outputs device [Bz,k+n_text,D], [Bz,k+n_text], [Bz,k+n_text].  T_in = n_vis + n_text.
 *   positions / idx_map (and their outputs) may be NULL together.  D*sizeof(dtype) must be a
 *   multiple of 16 bytes. */
int str_compact(str_ctx *ctx, int Bz, int T_in, int n_vis, int n_text, int k, int D, int dtype,
                const void *hidden, const int32_t *positions, const int32_t *idx_map,
                const int32_t *kept_idx, void *hidden_out, int32_t *positions_out,
                int32_t *idx_map_out, void *stream);

/* (5) Retention schedule -> keep counts (Section 3.2; appendix "Reduction Schedule
 * Configurations"; host only, no CUDA).  alpha_bp[l] is layer l's retention ratio in basis
 * points of the ORIGINAL visual count n0; K_out[l] = min(n_cur, max(min_keep, floor(alpha n0)))
 * is the visual count after layer l.  Layer l reduces iff K_out[l] < its incoming count. */
int str_schedule_keep_counts(const int *alpha_bp, int L, int n0, int min_keep, int *K_out);
/* Same for a stack whose layer kinds (STR_LAYER_*, host array [L]) are known: FFN layers never reduce, so a cut the
 * schedule places on an FFN layer is taken by the next Mamba / attention layer (K_out of an FFN layer equals its
 * incoming count).  The paper's all-layer schedules cut at Mamba and attention layers only. */
int str_schedule_keep_counts_layers(const int *alpha_bp, const int *layer_kinds, int L, int n0, int min_keep, int *K_out);
/* Sigmoid retention alpha_l = a_end + (a_start - a_end) * sigmoid(k (x0 - l/L)), in basis points
 * (rounded to nearest), l = 0..L-1.  Host only. */
int str_sigmoid_schedule_bp(int L, double k, double x0, double a_start, double a_end, int *alpha_bp_out);

/* (3') Density of an importance vector (Section 2, the sparsity analysis: "tokens needed for 80% of the importance
 * mass"): per row, the smallest k such that the k largest scores sum to at least mass_fraction of the row's total.
 * A diagnostic of how concentrated a layer's scores are; the mass-threshold dual of the rank threshold of (3).
 *   scores device [Bz,n_vis] fp32, all >= 0; mass_fraction in (0,1]; count_out device [Bz] int32 (0 for a row
 *   whose scores are all zero).  Sums are taken in fp64.  No workspace. */
int str_score_density(str_ctx *ctx, int Bz, int n_vis, const float *scores, float mass_fraction,
                      int32_t *count_out, void *stream);

/* ------------------------------------------------------------------------------------------
 * Block glue.  The paper gives only the recurrence and the scores; these are the standard
 * pre-norm Mamba-2 / GQA block pieces needed to run a layer stack.  Same conventions.
 * ------------------------------------------------------------------------------------------ */

/* out[M,N] = a[M,K] * w[N,K]^T (+ residual[M,N] if not NULL).  a, w, residual, out device, dtype.
 * Weights are stored [out_features, in_features] (K contiguous). */
size_t str_gemm_workspace_size(int M, int N, int K, int dtype);
int str_gemm(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
             const void *residual, void *out, void *workspace, size_t workspace_bytes, void *stream);

/* out[r,:] = in[r,:] / sqrt(mean(in[r,:]^2) + eps)  (unit weight), rows x D, dtype. */
int str_rmsnorm(str_ctx *ctx, int dtype, int rows, int D, float eps, const void *in, void *out,
                void *stream);

/* out[i] = max(in[i], 0)^2, n elements of dtype; out may equal in.  (Activation of the FFN block.) */
int str_relu_squared(str_ctx *ctx, int dtype, size_t n, const void *in, void *out, void *stream);

/* Mamba-2 pre-scan step on the in_proj output zxbcdt [Bz*T, 2*d_inner + 2*G*n + H] =
 * [z | x B C | dt_raw]: causal depthwise conv (width W, zero left padding per sequence, taps
 * conv_w [d_inner+2Gn, W] fp32, last tap on the current token, bias conv_b fp32) + SiLU on the
 * x B C columns, split into x_out [Bz,T,H,p], B_out, C_out [Bz,T,G,n] (dtype), and
 * dt_out [Bz,T,H] fp32 = softplus(dt_raw + dt_bias[h]). */
int str_mamba_conv_split(str_ctx *ctx, int dtype, int Bz, int T, int H, int p, int n, int G, int W,
                         const void *zxbcdt, const float *conv_w, const float *conv_b,
                         const float *dt_bias, void *x_out, void *B_out, void *C_out, float *dt_out,
                         void *stream);

/* The Mamba block's input side in one call: the in-projection followed by the pre-scan step above,
 * zxbcdt = u * w_in^T with u [Bz*T, D] (rows already normalised) and w_in [2*d_inner + 2*G*n + H, D], then
 * str_mamba_conv_split on it.  Where the tensor-core GEMM takes the shape (bf16, W = 4, d_inner and G*n
 * multiples of 32, H a multiple of 8, 16-byte aligned pointers) the conv, SiLU, split and softplus run in the
 * projection's epilogue, so the [x B C | dt] columns never make a round trip through memory; the results are
 * bit for bit those of the two separate calls, which is also what runs otherwise.
 *   zxbcdt  device [Bz*T, 2*d_inner + 2*G*n + H], dtype: on return its first d_inner columns hold the gate z;
 *           the other columns are scratch.  All other arguments as in str_gemm and str_mamba_conv_split.
 * Returns STR_ERR_INVALID_ARG on a null pointer or a non-positive size. */
int str_mamba_in_proj_conv(str_ctx *ctx, int dtype, int Bz, int T, int D, int H, int p, int n, int G, int W,
                           const void *u, const void *w_in, const float *conv_w, const float *conv_b,
                           const float *dt_bias, void *zxbcdt, void *x_out, void *B_out, void *C_out,
                           float *dt_out, void *stream);

/* out[r,:] = RMSNorm( y[r,:] * SiLU(z[r,:]) ) over d_inner columns; z is read in place from the
 * in_proj output (row stride ld_z elements, first d_inner columns). */
int str_gated_rmsnorm(str_ctx *ctx, int dtype, int rows, int d_inner, int ld_z, float eps,
                      const void *y, const void *z, void *out, void *stream);

/* Splits qkv [Bz*T, (Hq+2Hkv)*d] into q_out [Bz,T,Hq,d], k_out, v_out [Bz,T,Hkv,d] and applies
 * rotary embedding (half-split pairing (i, i+d/2), angle = position * theta^(-2i/d)) to q and k
 * using the carried original positions [Bz,T] int32. */
int str_rope_split(str_ctx *ctx, int dtype, int Bz, int T, int Hq, int Hkv, int d, float theta,
                   const int32_t *positions, const void *qkv, void *q_out, void *k_out,
                   void *v_out, void *stream);

/* Causal GQA softmax attention over each sequence: o[t] = sum_{j<=t} softmax_j(q_t.k_j*scale) v_j.
 * q,o device [Bz,T,Hq,d]; k,v device [Bz,T,Hkv,d]; dtype. */
typedef struct {
    int Bz, T, Hq, Hkv, d, dtype;
} str_attn_shape;
size_t str_attn_prefill_workspace_size(const str_attn_shape *s);
int str_attn_prefill(str_ctx *ctx, const str_attn_shape *s, const void *q, const void *k,
                     const void *v, float softmax_scale, void *o, void *workspace,
                     size_t workspace_bytes, void *stream);

/* The same attention for a gathered subset of the query rows (a layer that has selected its survivors before the
 * attention only needs their outputs; every incoming key and value is still attended to).  q_rows, o_rows device
 * [Bz,n_rows,Hq,d]; row_pos device [Bz,n_rows] int32, strictly ascending: the index of each query row in the key
 * sequence (row r attends to keys 0 .. row_pos[r]); NULL means rows 0 .. n_rows-1 with n_rows == T.  k, v device
 * [Bz,T,Hkv,d].  A row's output does not depend on which other rows are passed with it: it is bit-identical to the
 * row str_attn_prefill computes. */
int str_attn_prefill_rows(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q_rows, const int32_t *row_pos,
                          const void *k, const void *v, float softmax_scale, void *o_rows, void *workspace,
                          size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * Whole stack: token-reduced prefill with a per-layer keep schedule (Sections 3.1-3.2).
 * Layer l's mixer runs on the incoming tokens, its own importance score ranks the incoming
 * visual tokens, and its OUTPUT is compacted to keep_counts[l] visual tokens when that is
 * smaller than the incoming count.  Block wrapper: h <- h + Mixer(RMSNorm(h)).  FFN layers (the
 * hybrid's third block type, appendix "Models") only transform the rows they are given: their
 * keep count must equal the incoming count.
 * ------------------------------------------------------------------------------------------ */
enum { STR_LAYER_MAMBA = 0, STR_LAYER_ATTN = 1, STR_LAYER_FFN = 2 };
enum { STR_SCORE_DECOUPLED = 0, STR_SCORE_FULL_DYNAMIC = 1 };
typedef struct {
    int kind;             /* STR_LAYER_MAMBA, STR_LAYER_ATTN or STR_LAYER_FFN                   */
    const void *w_in;     /* device: Mamba in_proj [2*d_inner+2Gn+H, D] | attention W_qkv [(Hq+2Hkv)d, D] | FFN W_up [ffn_dim, D] */
    const void *w_out;    /* device: Mamba out_proj [D, d_inner]        | attention W_o [D, Hq*d]         | FFN W_down [D, ffn_dim] */
    const float *conv_w;  /* device, Mamba only: [d_inner+2Gn, W]                                */
    const float *conv_b;  /* device, Mamba only: [d_inner+2Gn]                                   */
    const float *dt_bias; /* device, Mamba only: [H]                                             */
    const float *A;       /* device, Mamba only: [H], negative                                   */
} str_layer;
typedef struct {
    int Bz, n_vis, n_text, D, dtype;
    int H, p, n, G, Q, conv_width;     /* Mamba-2 layer shape     */
    int Hq, Hkv, d;                    /* attention layer shape   */
    float rope_theta, norm_eps;
    int n_layers;
    const str_layer *layers;           /* host array [n_layers]                              */
    const int *keep_counts;            /* host array [n_layers], from str_schedule_keep_counts */
    int score_every_layer;             /* nonzero: also compute (not apply) the score at layers that do not reduce */
    int mamba_score_kind;              /* STR_SCORE_DECOUPLED (Eq. 2, the method) or STR_SCORE_FULL_DYNAMIC (Eq. 1, its ablation) */
    int attn_score_denominator;        /* STR_ATTN_DENOM_VISUAL (the paper's formula) or STR_ATTN_DENOM_CAUSAL_ROW */
    int ffn_dim;                       /* width of the FFN layers, h <- h + W_down relu(W_up RMSNorm(h))^2; they never score or reduce */
} str_stack_desc;
size_t str_stack_workspace_size(const str_stack_desc *d);
/* hidden_in device [Bz, n_vis+n_text, D] dtype.  Outputs (device): hidden_out
 * [Bz, K_last+n_text, D] dtype, positions_out / idx_map_out [Bz, K_last+n_text] int32 (original
 * token ids of the surviving rows), where K_last = keep_counts[n_layers-1].
 * kept_trace (device, optional, may be NULL): for each reducing layer in order, its kept
 * indices [Bz,K_l] int32, packed one after the other; scores_trace likewise [Bz,n_cur] fp32. */
int str_stack_prefill(str_ctx *ctx, const str_stack_desc *d, const void *hidden_in,
                      void *hidden_out, int32_t *positions_out, int32_t *idx_map_out,
                      int32_t *kept_trace, float *scores_trace, void *workspace,
                      size_t workspace_bytes, void *stream);
/* Optional inputs and outputs of the stack, for callers that continue from a reduced context or hand the result to
 * a decoder (Section 2 "stateful compression": the tokens a Mamba layer drops stay absorbed in its state; later steps
 * run on the kept set).  Every pointer is a device pointer owned by the caller and may be NULL.
 *   positions_in / idx_map_in [Bz, n_vis+n_text] int32: original token ids of the incoming rows (strictly ascending per
 *     sequence); NULL means 0 .. n_vis+n_text-1.  positions_in feeds the rotary embedding, idx_map_in is carried
 *     through the compactions into idx_map_out.
 *   mamba_final_states: for each Mamba layer, in layer order, the recurrent state after the last incoming token,
 *     [Bz,H,p,n] fp32, packed one after the other.
 *   attn_k_out / attn_v_out: for each attention layer, in layer order, the post-RoPE keys / the values of the rows that
 *     LEAVE the layer (the kept visual rows, then the text rows), [Bz, K_l+n_text, Hkv, d] dtype, packed one after the
 *     other; attn_pos_out likewise [Bz, K_l+n_text] int32 holds their original positions. */
typedef struct {
    const int32_t *positions_in;
    const int32_t *idx_map_in;
    float *mamba_final_states;
    void *attn_k_out;
    void *attn_v_out;
    int32_t *attn_pos_out;
} str_stack_io;
/* str_stack_prefill with the optional inputs / outputs above (io == NULL: exactly str_stack_prefill). */
int str_stack_prefill_ex(str_ctx *ctx, const str_stack_desc *d, const str_stack_io *io, const void *hidden_in,
                         void *hidden_out, int32_t *positions_out, int32_t *idx_map_out, int32_t *kept_trace,
                         float *scores_trace, void *workspace, size_t workspace_bytes, void *stream);
/* Same, with HOST hidden_in / hidden_out / idx_map_out buffers (pinned memory recommended):
 * copies the input to the device, runs the stack, copies the results back, and synchronises
 * `stream` before returning.  The device staging area is part of the workspace
 * (str_stack_host_workspace_size).  The input travels in a few row blocks on a copy stream owned
 * by the context (created on the first call), so that the first layer starts on block 0 while the
 * rest is still in flight, and the last layer's output projection is issued in row blocks, each
 * copied back while the next is computed; a context therefore serves one such call at a time. */
size_t str_stack_host_workspace_size(const str_stack_desc *d);
int str_stack_prefill_host(str_ctx *ctx, const str_stack_desc *d, const void *hidden_in_host,
                           void *hidden_out_host, int32_t *idx_map_out_host, void *workspace,
                           size_t workspace_bytes, void *stream);

/* Optional device timing by kernel category.  While enabled, every leaf entry point records a CUDA
 * event pair around its launches on the caller's stream (str_profile_enable allocates events lazily on
 * first use).  str_profile_collect synchronises on the recorded events, adds the elapsed milliseconds
 * and the number of calls per category into the caller's host arrays (n >= STR_PROF_CATEGORIES) and
 * forgets the recorded spans.  Categories: 0 GEMM, 1 Mamba-2 scan, 2 Mamba importance, 3 attention
 * importance, 4 top-K select, 5 compaction, 6 attention forward, 7 element-wise glue. */
#define STR_PROF_CATEGORIES 8
int str_profile_enable(str_ctx *ctx, int on);
int str_profile_collect(str_ctx *ctx, double *ms_by_category, long long *calls_by_category, int n);

/* Number of kernels this library has launched on this context since creation (host counter). */
long long str_launch_count(const str_ctx *ctx);
/* How many entry-point calls on this context ran a tensor-core (tcgen05) kernel and how many fell back to the plain
 * fp32-FMA kernel of the same entry point (shapes or dtypes the tensor-core kernels do not tile, or
 * STR_FORCE_SIMT=1 in the environment).  Counted for the scan, the three scores, the GEMM and the attention forward. */
int str_path_counts(const str_ctx *ctx, long long *tensor_core_calls, long long *fallback_calls);
/* Self-test of the bounded device-side waits: launches one CTA that waits on a barrier nobody signals, gives up
 * after probe_limit probes (1 .. 2^20), records STR_ERR_TIMEOUT in the status word and returns normally.  The next
 * str_check_status reports the timeout once and clears it.  No tensor memory, no copies: safe at any time. */
int str_selftest_wait_timeout(str_ctx *ctx, unsigned int probe_limit, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STR_H_ */
