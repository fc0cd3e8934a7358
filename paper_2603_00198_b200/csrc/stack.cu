// str_stack_prefill: token-reduced prefill of a hybrid Mamba-2 / attention layer stack.
// Host loop over layers; every step is a kernel of this library enqueued on one stream, with no
// device->host synchronisation in between (the keep counts are known in advance because the
// schedule does not depend on the input).
#include <string.h>

#include <stdlib.h>

#include "dispatch.cuh"

// Debug switch: STR_CONV_FUSE=0 keeps the pre-scan step in its own kernel (A/B runs of the fused epilogue).  Read at
// every call, so that one process can run both routes.
static bool str_conv_fusion_on() {
    const char *e = getenv("STR_CONV_FUSE");
    return !(e && e[0] == '0');
}

namespace {

__global__ void iota_rows_kernel(int rows, int T, int32_t *a, int32_t *b) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < rows) { a[i] = i % T; b[i] = i % T; }
}

// Index in the incoming sequence of every row that survives a cut: the kept visual rows, then the text rows.
__global__ void survivor_rows_kernel(int Bz, int n_vis, int n_text, int k, const int32_t *__restrict__ kept,
                                     int32_t *__restrict__ rows_out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Bz * (k + n_text)) return;
    const int b = i / (k + n_text), j = i % (k + n_text);
    rows_out[i] = j < k ? kept[(size_t)b * k + j] : n_vis + (j - k);
}

// Rows of a small fp32 side array (the partial sums of squares of the hidden rows) for the rows that survive a cut.
__global__ void gather_rows_f32_kernel(int Bz, int T_in, int n_vis, int n_text, int k, int width, const int32_t *__restrict__ kept,
                                       const float *__restrict__ in, float *__restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Bz * (k + n_text) * width) return;
    const int c = i % width, r = i / width;
    const int b = r / (k + n_text), j = r % (k + n_text);
    const int src = j < k ? kept[(size_t)b * k + j] : n_vis + (j - k);
    out[i] = in[((size_t)b * T_in + src) * width + c];
}

struct Regions {
    size_t hidden[2], normed, proj, bufA, bufB, bufC, bufY, dt, pos[2], idx[2], scores, kept, rowpos, ss[3], sub, total;
    size_t sub_bytes;
};

inline size_t imax(size_t a, size_t b) { return a > b ? a : b; }

bool desc_ok(const str_stack_desc *d) {
    if (!d || d->Bz <= 0 || d->n_vis < 0 || d->n_text <= 0 || d->D <= 0 || d->n_layers <= 0 || !d->layers ||
        !d->keep_counts || (d->dtype != STR_F32 && d->dtype != STR_BF16) ||
        (d->mamba_score_kind != STR_SCORE_DECOUPLED && d->mamba_score_kind != STR_SCORE_FULL_DYNAMIC) ||
        (d->attn_score_denominator != STR_ATTN_DENOM_VISUAL && d->attn_score_denominator != STR_ATTN_DENOM_CAUSAL_ROW))
        return false;
    bool has_m = false, has_a = false;
    int n_cur = d->n_vis;
    for (int l = 0; l < d->n_layers; ++l) {
        const str_layer &L = d->layers[l];
        if (L.kind == STR_LAYER_MAMBA) {
            has_m = true;
            if (!L.w_in || !L.w_out || !L.conv_w || !L.conv_b || !L.dt_bias || !L.A) return false;
        } else if (L.kind == STR_LAYER_ATTN) {
            has_a = true;
            if (!L.w_in || !L.w_out) return false;
        } else if (L.kind == STR_LAYER_FFN) {
            if (!L.w_in || !L.w_out || d->ffn_dim <= 0 || d->keep_counts[l] != n_cur) return false;
        } else {
            return false;
        }
        if (d->keep_counts[l] < 0 || d->keep_counts[l] > n_cur) return false;
        n_cur = d->keep_counts[l];
    }
    if (has_m && (d->H <= 0 || d->p <= 0 || d->n <= 0 || d->G <= 0 || d->H % d->G != 0 || d->conv_width <= 0))
        return false;
    if (has_a && (d->Hq <= 0 || d->Hkv <= 0 || d->Hq % d->Hkv != 0 || d->d <= 0 || (d->d & 1) || d->rope_theta <= 0.f))
        return false;
    return true;
}

Regions plan(const str_stack_desc *d) {
    Regions r;
    const size_t e = dtype_size(d->dtype);
    const size_t T0 = (size_t)d->n_vis + d->n_text, R = (size_t)d->Bz * T0;
    bool has_m = false, has_a = false;
    bool has_f = false;
    for (int l = 0; l < d->n_layers; ++l) {
        const int kind = d->layers[l].kind;
        (kind == STR_LAYER_MAMBA ? has_m : kind == STR_LAYER_ATTN ? has_a : has_f) = true;
    }
    const size_t dff = has_f ? (size_t)d->ffn_dim : 0;
    const size_t d_inner = has_m ? (size_t)d->H * d->p : 0, gn = has_m ? (size_t)d->G * d->n : 0;
    const size_t dip = has_m ? 2 * d_inner + 2 * gn + d->H : 0;
    const size_t qd = has_a ? (size_t)d->Hq * d->d : 0, kd = has_a ? (size_t)d->Hkv * d->d : 0;
    const size_t dqkv = qd + 2 * kd;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
    r.hidden[0] = take(R * d->D * e);
    r.hidden[1] = take(R * d->D * e);
    r.normed = take(R * d->D * e);
    r.proj = take(R * imax(imax(dip, dqkv), dff) * e);
    r.bufA = take(R * imax(d_inner, qd) * e);
    r.bufB = take(R * imax(gn, kd) * e);
    r.bufC = take(R * imax(gn, kd) * e);
    r.bufY = take(R * imax(d_inner, qd) * e);
    r.dt = take(R * (has_m ? d->H : 1) * sizeof(float));
    for (int i = 0; i < 2; ++i) { r.pos[i] = take(R * 4); r.idx[i] = take(R * 4); }
    r.scores = take((size_t)d->Bz * imax(d->n_vis, 1) * 4);
    r.kept = take((size_t)d->Bz * imax(d->n_vis, 1) * 4);
    r.rowpos = take(R * 4);
    for (int i = 0; i < 3; ++i) r.ss[i] = take(R * str_ss_blocks(d->D) * sizeof(float));
    size_t sub = 0;
    if (has_m) {
        str_ssd_shape s = {d->Bz, (int)T0, d->H, d->p, d->n, d->G, d->Q, d->dtype};
        sub = imax(sub, str_mamba2_prefill_workspace_size(&s));
        str_ssm_score_shape ss = {d->Bz, (int)T0, d->H, d->n, d->G, d->dtype};
        sub = imax(sub, str_mamba_importance_workspace_size(&ss, d->n_vis, d->n_text));
        if (d->mamba_score_kind == STR_SCORE_FULL_DYNAMIC)
            sub = imax(sub, str_mamba_importance_dynamic_workspace_size(&ss, d->n_vis, d->n_text));
        sub = imax(sub, str_gemm_workspace_size((int)R, (int)dip, d->D, d->dtype));
    }
    if (has_a) {
        str_attn_score_shape as = {d->Bz, (int)T0, d->Hq, d->Hkv, d->d, d->dtype};
        sub = imax(sub, str_attn_importance_workspace_size(&as, d->n_vis, d->n_text));
        str_attn_shape at = {d->Bz, (int)T0, d->Hq, d->Hkv, d->d, d->dtype};
        sub = imax(sub, str_attn_prefill_workspace_size(&at));
        sub = imax(sub, str_gemm_workspace_size((int)R, (int)dqkv, d->D, d->dtype));
    }
    if (has_f) sub = imax(sub, str_gemm_workspace_size((int)R, (int)dff, d->D, d->dtype));
    sub = imax(sub, str_topk_select_workspace_size(d->Bz, d->n_vis, d->n_vis));
    r.sub_bytes = align_up(sub, 256);
    r.sub = take(r.sub_bytes);
    r.total = off;
    return r;
}

}  // namespace

extern "C" size_t str_stack_workspace_size(const str_stack_desc *d) {
    if (!desc_ok(d)) return 0;
    return plan(d).total;
}

// Input feed of the host-buffer entry point: the hidden states arrive in `chunks` row blocks of `rows_per_chunk`
// rows, block j being complete once `ready[j]` has fired.  Only the first layer's norm and first projection read
// the input row by row, so only they are issued per block.
// Output drain: the last layer's output projection is issued in `out_chunks` row blocks; after each block an event is
// recorded on the caller's stream and the block is copied to the host on `copy_stream`, so that only the last block's
// copy is exposed.
struct StackFeed {
    int chunks; int rows_per_chunk; cudaEvent_t *ready;
    int out_chunks; cudaEvent_t *out_done; cudaStream_t copy_stream; void *out_host;
};

#define STR_TRY(call)              \
    do {                           \
        int _rc = (call);          \
        if (_rc != STR_OK) return _rc; \
    } while (0)

static int stack_prefill_impl(str_ctx *ctx, const str_stack_desc *d, const str_stack_io *io, const void *hidden_in, void *hidden_out,
                              int32_t *positions_out, int32_t *idx_map_out, int32_t *kept_trace, float *scores_trace,
                              void *workspace, size_t workspace_bytes, void *stream, const StackFeed *feed) {
    if (!ctx || !desc_ok(d) || !hidden_in || !hidden_out || !workspace) return STR_ERR_INVALID_ARG;
    if (((uintptr_t)workspace & 255) != 0) return STR_ERR_INVALID_ARG;
    const Regions r = plan(d);
    if (workspace_bytes < r.total) return STR_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    const int Bz = d->Bz, M = d->n_text, D = d->D, dtype = d->dtype;
    void *hid[2] = {ws + r.hidden[0], ws + r.hidden[1]};
    int32_t *pos[2] = {(int32_t *)(ws + r.pos[0]), (int32_t *)(ws + r.pos[1])};
    int32_t *idx[2] = {(int32_t *)(ws + r.idx[0]), (int32_t *)(ws + r.idx[1])};
    void *normed = ws + r.normed, *proj = ws + r.proj, *bufA = ws + r.bufA, *bufB = ws + r.bufB;
    void *bufC = ws + r.bufC, *bufY = ws + r.bufY, *sub = ws + r.sub;
    float *dt = (float *)(ws + r.dt);
    float *scores_int = (float *)(ws + r.scores);
    int32_t *kept_int = (int32_t *)(ws + r.kept);

    int n_cur = d->n_vis;
    {
        const int rows = Bz * (n_cur + M);
        iota_rows_kernel<<<ceil_div(rows, 256), 256, 0, st>>>(rows, n_cur + M, pos[0], idx[0]);
        STR_TRY(str_launch_ok(ctx));
        // a caller that continues from a reduced context brings the original token ids of its rows
        if (io && io->positions_in)
            STR_CUDA_OK(cudaMemcpyAsync(pos[0], io->positions_in, (size_t)rows * 4, cudaMemcpyDeviceToDevice, st));
        if (io && io->idx_map_in)
            STR_CUDA_OK(cudaMemcpyAsync(idx[0], io->idx_map_in, (size_t)rows * 4, cudaMemcpyDeviceToDevice, st));
    }
    float *fs_out = io ? io->mamba_final_states : nullptr;
    char *k_out = io ? (char *)io->attn_k_out : nullptr, *v_out = io ? (char *)io->attn_v_out : nullptr;
    int32_t *kvpos_out = io ? io->attn_pos_out : nullptr;
    const void *cur = hidden_in;
    int hsel = 0;      // next free hidden buffer
    int psel = 0;      // current positions / idx buffer
    // The RMSNorm in front of every layer is fused into the layer's first projection: the projection runs on the hidden
    // rows themselves and scales its output rows by 1/rms, taken from partial sums of squares that the previous layer's
    // last projection left behind (for the stack's input: from one pass over it).  `normed` is only a scratch buffer
    // for the survivors' residual rows now.
    const int ntD = str_ss_blocks(D);
    const float inv_D = 1.0f / (float)D;
    float *ssb[3] = {(float *)(ws + r.ss[0]), (float *)(ws + r.ss[1]), (float *)(ws + r.ss[2])};
    const float *cur_ss = ssb[0];
    int ssel = 1;      // next free buffer of partial sums
    if (!feed) STR_TRY(str_row_sumsq(ctx, dtype, Bz * (n_cur + M), D, hidden_in, ssb[0], stream));
    size_t kept_off = 0, score_off = 0;

    for (int l = 0; l < d->n_layers; ++l) {
        const str_layer &L = d->layers[l];
        const int T = n_cur + M, rows = Bz * T;
        const int K = d->keep_counts[l];
        const bool reduce = K < n_cur;
        const bool last = l == d->n_layers - 1;
        const bool want_score = reduce || d->score_every_layer;
        float *scores = (reduce && scores_trace) ? scores_trace + score_off : scores_int;
        int32_t *kept = (reduce && kept_trace) ? kept_trace + kept_off : kept_int;
        void *mix_out = (last && !reduce) ? hidden_out : hid[hsel];

        // the layer's first projection with the RMSNorm of the layer input fused in: [rows x N] = RMSNorm(cur) W^T into `proj`
        // With `conv` (a Mamba layer) the projection's epilogue also runs the pre-scan step when the shapes allow;
        // *conv_fused tells the caller which of the two follow-up kernels is due.
        auto norm_and_project = [&](int N, const void *w, const StrConvEpilogue *conv = nullptr, bool *conv_fused = nullptr) -> int {
            const bool fed = feed && l == 0;
            const int step = fed ? feed->rows_per_chunk : rows;
            const size_t esz = dtype_size(dtype);
            const bool fuse = conv && !str_force_simt() && str_conv_fusion_on() && step % 32 == 0 &&
                              str_gemm_conv_supported(dtype, rows < step ? rows : step, N, D, cur, w, proj, *conv);
            if (conv_fused) *conv_fused = fuse;
            for (int j = 0, r0 = 0; r0 < rows; ++j, r0 += step) {
                const int nr = rows - r0 < step ? rows - r0 : step;
                float *ss_blk = ssb[0] + (size_t)r0 * ntD;
                if (fed) {
                    STR_CUDA_OK(cudaStreamWaitEvent(st, feed->ready[j], 0));
                    STR_TRY(str_row_sumsq(ctx, dtype, nr, D, (const char *)cur + (size_t)r0 * D * esz, ss_blk, stream));
                }
                const StrRowNorm rn = {cur_ss + (size_t)r0 * ntD, ntD, inv_D, d->norm_eps, nullptr};
                if (fuse) {
                    StrProfScope prof_scope(ctx, STR_CAT_GEMM, stream);
                    StrConvEpilogue cv = *conv;
                    cv.row_base = r0;
                    ++ctx->tc_calls;
                    STR_TRY(str_gemm_tc(ctx, nr, N, D, (const char *)cur + (size_t)r0 * D * esz, w, nullptr,
                                        (char *)proj + (size_t)r0 * N * esz, rn, cv, st));
                    continue;
                }
                STR_TRY(str_gemm_fused(ctx, dtype, nr, N, D, (const char *)cur + (size_t)r0 * D * esz, w, nullptr,
                                       (char *)proj + (size_t)r0 * N * esz, rn, stream));
            }
            return STR_OK;
        };
        // the layer's last projection adds the residual and leaves the partial sums of squares of its output rows for
        // the next layer's fused norm
        float *next_ss = last ? nullptr : ssb[ssel];
        auto project_out = [&](int nrows, int K_in, const void *a, const void *w, const void *residual, void *out_rows) -> int {
            const StrRowNorm rn = {nullptr, 0, 0.f, 0.f, next_ss};
            if (!(last && feed && feed->out_chunks > 1))
                return str_gemm_fused(ctx, dtype, nrows, D, K_in, a, w, residual, out_rows, rn, stream);
            // host-buffer call, last layer: row blocks (whole GEMM row tiles), each copied out as soon as it is done
            const size_t esz = dtype_size(dtype);
            const int step = (int)align_up((size_t)ceil_div(nrows, feed->out_chunks), 128);
            for (int j = 0, r0 = 0; r0 < nrows; ++j, r0 += step) {
                const int nr = nrows - r0 < step ? nrows - r0 : step;
                STR_TRY(str_gemm_fused(ctx, dtype, nr, D, K_in, (const char *)a + (size_t)r0 * K_in * esz, w,
                                       (const char *)residual + (size_t)r0 * D * esz, (char *)out_rows + (size_t)r0 * D * esz, rn,
                                       stream));
                STR_CUDA_OK(cudaEventRecord(feed->out_done[j], st));
                STR_CUDA_OK(cudaStreamWaitEvent(feed->copy_stream, feed->out_done[j], 0));
                STR_CUDA_OK(cudaMemcpyAsync((char *)feed->out_host + (size_t)r0 * D * esz, (const char *)out_rows + (size_t)r0 * D * esz,
                                            (size_t)nr * D * esz, cudaMemcpyDeviceToHost, feed->copy_stream));
            }
            return STR_OK;
        };
        // A reducing layer selects BEFORE the mixer's epilogue: the score only needs the projections, so the rows
        // about to be dropped skip the gate / norm / output projection (their inputs still feed the scan state
        // and the attention keys).  The surviving rows come out bit-identical to computing every row first.
        void *dst = !reduce ? mix_out : (last ? hidden_out : hid[hsel]);
        int32_t *pdst = (last && positions_out) ? positions_out : pos[1 - psel];
        int32_t *idst = (last && idx_map_out) ? idx_map_out : idx[1 - psel];
        const int rows_out = reduce ? Bz * (K + M) : rows;
        if (L.kind == STR_LAYER_MAMBA) {
            const int d_inner = d->H * d->p, gn = d->G * d->n, dip = 2 * d_inner + 2 * gn + d->H;
            // conv + SiLU + split + softplus(dt) ride in the in-projection's epilogue when the kernel supports the shape
            StrConvEpilogue conv = {d->conv_width == 4 ? T : 0, 0, reduce ? 0 : d_inner, d_inner, gn, d->H, L.conv_w, L.conv_b,
                                    L.dt_bias, (__nv_bfloat16 *)bufA, (__nv_bfloat16 *)bufB, (__nv_bfloat16 *)bufC, dt};
            bool conv_fused = false;
            if (reduce) {
                // the gate z is only needed for the rows that survive: project [x B C | dt] for every row now (the
                // weight rows after the first d_inner) and z for the kept rows after the selection
                const char *w_rest = (const char *)L.w_in + (size_t)d_inner * D * dtype_size(dtype);
                STR_TRY(norm_and_project(dip - d_inner, w_rest, &conv, &conv_fused));
            } else {
                STR_TRY(norm_and_project(dip, L.w_in, &conv, &conv_fused));
            }
            if (conv_fused)
                STR_TRY(str_mamba_conv_edge_rows(ctx, Bz, T, conv.zoff + d_inner + 2 * gn + d->H, conv, proj, stream));
            else
                STR_TRY(str_mamba_conv_split_rows(ctx, dtype, Bz, T, d->H, d->p, d->n, d->G, d->conv_width, !reduce, proj,
                                                  L.conv_w, L.conv_b, L.dt_bias, bufA, bufB, bufC, dt, stream));
            str_ssd_shape s = {Bz, T, d->H, d->p, d->n, d->G, d->Q, dtype};
            STR_TRY(str_mamba2_prefill(ctx, &s, bufA, dt, L.A, bufB, bufC, nullptr, nullptr, bufY, fs_out, sub,
                                       r.sub_bytes, stream));
            if (fs_out) fs_out += (size_t)Bz * d->H * d->p * d->n;
            if (want_score && n_cur > 0) {
                str_ssm_score_shape ss = {Bz, T, d->H, d->n, d->G, dtype};
                if (d->mamba_score_kind == STR_SCORE_FULL_DYNAMIC)
                    STR_TRY(str_mamba_importance_dynamic(ctx, &ss, n_cur, M, bufB, bufC, dt, L.A, scores, sub, r.sub_bytes, stream));
                else
                    STR_TRY(str_mamba_importance(ctx, &ss, n_cur, M, bufB, bufC, dt, scores, sub, r.sub_bytes, stream));
            }
            if (reduce) {
                STR_TRY(str_topk_select(ctx, Bz, n_cur, K, scores, kept, sub, r.sub_bytes, stream));
                // hidden rows (the residual), positions and the index map of the survivors, and their sums of squares
                STR_TRY(str_compact(ctx, Bz, T, n_cur, M, K, D, dtype, cur, pos[psel], idx[psel], kept, normed, pdst, idst,
                                    stream));
                float *ss_kept = ssb[2];
                gather_rows_f32_kernel<<<ceil_div(rows_out * ntD, 256), 256, 0, st>>>(Bz, T, n_cur, M, K, ntD, kept, cur_ss, ss_kept);
                STR_TRY(str_launch_ok(ctx));
                // z of the survivors: the same gathered hidden rows, projected with the first d_inner weight rows (and
                // the fused norm) into the projection buffer, whose [x B C | dt] content was consumed by the conv
                const StrRowNorm rnz = {ss_kept, ntD, inv_D, d->norm_eps, nullptr};
                STR_TRY(str_gemm_fused(ctx, dtype, rows_out, d_inner, D, normed, L.w_in, nullptr, proj, rnz, stream));
                STR_TRY(str_gated_rmsnorm_gather(ctx, dtype, Bz, T, n_cur, M, K, d_inner, d_inner, d->norm_eps, bufY, proj, true,
                                                 kept, bufA, stream));
                STR_TRY(project_out(rows_out, d_inner, bufA, L.w_out, normed, dst));
            } else {
                STR_TRY(str_gated_rmsnorm(ctx, dtype, rows, d_inner, dip, d->norm_eps, bufY, proj, bufA, stream));
                STR_TRY(project_out(rows, d_inner, bufA, L.w_out, cur, dst));
            }
        } else if (L.kind == STR_LAYER_FFN) {
            // h <- h + W_down relu(W_up RMSNorm(h))^2; the activation runs in place on the up-projection
            const int F = d->ffn_dim;
            STR_TRY(norm_and_project(F, L.w_in));
            STR_TRY(str_relu_squared(ctx, dtype, (size_t)rows * F, proj, proj, stream));
            STR_TRY(project_out(rows, F, proj, L.w_out, cur, dst));
        } else {
            const int qd = d->Hq * d->d, kd = d->Hkv * d->d;
            STR_TRY(norm_and_project(qd + 2 * kd, L.w_in));
            STR_TRY(str_rope_split(ctx, dtype, Bz, T, d->Hq, d->Hkv, d->d, d->rope_theta, pos[psel], proj, bufA, bufB,
                                   bufC, stream));
            str_attn_shape as = {Bz, T, d->Hq, d->Hkv, d->d, dtype};
            const float scale = 1.0f / sqrtf((float)d->d);
            if (want_score && n_cur > 0) {
                str_attn_score_shape ss = {Bz, T, d->Hq, d->Hkv, d->d, dtype};
                STR_TRY(str_attn_importance_ex(ctx, &ss, n_cur, M, bufA, bufB, scale, d->attn_score_denominator, scores, sub,
                                               r.sub_bytes, stream));
            }
            if (reduce) {
                // The score needs the text queries and the keys only, so the layer selects first and runs the attention
                // for the surviving query rows alone, against every incoming key and value.
                STR_TRY(str_topk_select(ctx, Bz, n_cur, K, scores, kept, sub, r.sub_bytes, stream));
                STR_TRY(str_compact(ctx, Bz, T, n_cur, M, K, D, dtype, cur, pos[psel], idx[psel], kept, normed, pdst, idst,
                                    stream));
                // the survivors' queries go to the projection buffer (its q | k | v content has been split out)
                STR_TRY(str_compact(ctx, Bz, T, n_cur, M, K, qd, dtype, bufA, nullptr, nullptr, kept, proj, nullptr, nullptr,
                                    stream));
                int32_t *rowpos = (int32_t *)(ws + r.rowpos);
                survivor_rows_kernel<<<ceil_div(rows_out, 256), 256, 0, st>>>(Bz, n_cur, M, K, kept, rowpos);
                STR_TRY(str_launch_ok(ctx));
                STR_TRY(str_attn_prefill_rows(ctx, &as, K + M, proj, rowpos, bufB, bufC, scale, bufY, sub, r.sub_bytes, stream));
                STR_TRY(project_out(rows_out, qd, bufY, L.w_out, normed, dst));
            } else {
                STR_TRY(str_attn_prefill(ctx, &as, bufA, bufB, bufC, scale, bufY, sub, r.sub_bytes, stream));
                STR_TRY(project_out(rows, qd, bufY, L.w_out, cur, dst));
            }
            // hand-off to a decoder: keys, values and positions of the rows that leave the layer
            if (k_out || v_out || kvpos_out) {
                const size_t kv_bytes = (size_t)rows_out * kd * dtype_size(dtype);
                if (reduce) {
                    if (k_out) STR_TRY(str_compact(ctx, Bz, T, n_cur, M, K, kd, dtype, bufB, nullptr, nullptr, kept, k_out, nullptr, nullptr, stream));
                    if (v_out) STR_TRY(str_compact(ctx, Bz, T, n_cur, M, K, kd, dtype, bufC, nullptr, nullptr, kept, v_out, nullptr, nullptr, stream));
                    if (kvpos_out) STR_CUDA_OK(cudaMemcpyAsync(kvpos_out, pdst, (size_t)rows_out * 4, cudaMemcpyDeviceToDevice, st));
                } else {
                    if (k_out) STR_CUDA_OK(cudaMemcpyAsync(k_out, bufB, kv_bytes, cudaMemcpyDeviceToDevice, st));
                    if (v_out) STR_CUDA_OK(cudaMemcpyAsync(v_out, bufC, kv_bytes, cudaMemcpyDeviceToDevice, st));
                    if (kvpos_out) STR_CUDA_OK(cudaMemcpyAsync(kvpos_out, pos[psel], (size_t)rows_out * 4, cudaMemcpyDeviceToDevice, st));
                }
                if (k_out) k_out += kv_bytes;
                if (v_out) v_out += kv_bytes;
                if (kvpos_out) kvpos_out += rows_out;
            }
        }
        cur = dst;
        if (next_ss) { cur_ss = next_ss; ssel = (next_ss == ssb[0]) ? 1 : 0; }
        if (dst == hid[0]) hsel = 1;
        else if (dst == hid[1]) hsel = 0;
        if (reduce) {
            psel = 1 - psel;
            kept_off += (size_t)Bz * K;
            score_off += (size_t)Bz * n_cur;
            n_cur = K;
            if (last) return STR_OK;          // positions / index map already written where the caller wants them
        }
    }
    // last layer did not reduce: hidden_out holds the result; hand back the carried ids
    const size_t nb = (size_t)Bz * (n_cur + M) * 4;
    if (positions_out) STR_CUDA_OK(cudaMemcpyAsync(positions_out, pos[psel], nb, cudaMemcpyDeviceToDevice, st));
    if (idx_map_out) STR_CUDA_OK(cudaMemcpyAsync(idx_map_out, idx[psel], nb, cudaMemcpyDeviceToDevice, st));
    return STR_OK;
}

extern "C" int str_stack_prefill(str_ctx *ctx, const str_stack_desc *d, const void *hidden_in, void *hidden_out,
                                 int32_t *positions_out, int32_t *idx_map_out, int32_t *kept_trace,
                                 float *scores_trace, void *workspace, size_t workspace_bytes, void *stream) {
    return stack_prefill_impl(ctx, d, nullptr, hidden_in, hidden_out, positions_out, idx_map_out, kept_trace, scores_trace,
                              workspace, workspace_bytes, stream, nullptr);
}

extern "C" int str_stack_prefill_ex(str_ctx *ctx, const str_stack_desc *d, const str_stack_io *io, const void *hidden_in,
                                    void *hidden_out, int32_t *positions_out, int32_t *idx_map_out, int32_t *kept_trace,
                                    float *scores_trace, void *workspace, size_t workspace_bytes, void *stream) {
    return stack_prefill_impl(ctx, d, io, hidden_in, hidden_out, positions_out, idx_map_out, kept_trace, scores_trace,
                              workspace, workspace_bytes, stream, nullptr);
}

extern "C" size_t str_stack_host_workspace_size(const str_stack_desc *d) {
    if (!desc_ok(d)) return 0;
    const size_t e = dtype_size(d->dtype);
    const size_t Rin = (size_t)d->Bz * ((size_t)d->n_vis + d->n_text);
    const size_t Rout = (size_t)d->Bz * ((size_t)d->keep_counts[d->n_layers - 1] + d->n_text);
    return align_up(Rin * d->D * e, 256) + align_up(Rout * d->D * e, 256) + 2 * align_up(Rout * 4, 256) + plan(d).total;
}

extern "C" int str_stack_prefill_host(str_ctx *ctx, const str_stack_desc *d, const void *hidden_in_host,
                                      void *hidden_out_host, int32_t *idx_map_out_host, void *workspace,
                                      size_t workspace_bytes, void *stream) {
    if (!ctx || !desc_ok(d) || !hidden_in_host || !hidden_out_host || !workspace) return STR_ERR_INVALID_ARG;
    if (workspace_bytes < str_stack_host_workspace_size(d)) return STR_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t e = dtype_size(d->dtype);
    const size_t Rin = (size_t)d->Bz * ((size_t)d->n_vis + d->n_text);
    const size_t Rout = (size_t)d->Bz * ((size_t)d->keep_counts[d->n_layers - 1] + d->n_text);
    char *ws = (char *)workspace;
    void *in_dev = ws;  ws += align_up(Rin * d->D * e, 256);
    void *out_dev = ws; ws += align_up(Rout * d->D * e, 256);
    int32_t *pos_dev = (int32_t *)ws; ws += align_up(Rout * 4, 256);
    int32_t *idx_dev = (int32_t *)ws; ws += align_up(Rout * 4, 256);
    // The input is copied in a few row blocks on a stream of the context's own, so that the first layer's norm and
    // projection of block j run while block j+1 is still on its way (pinned host memory makes the copies
    // asynchronous; with pageable memory they simply serialise).  Stream and events are created on first use.
    constexpr int CHUNKS = 8, OUT_CHUNKS = 4;
    if (!ctx->copy_stream) {
        STR_CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 18; ++i) STR_CUDA_OK(cudaEventCreateWithFlags(&ctx->copy_ev[i], cudaEventDisableTiming));
    }
    const size_t per = align_up((Rin + CHUNKS - 1) / CHUNKS, 128);          // rows per block: whole GEMM row tiles
    STR_CUDA_OK(cudaEventRecord(ctx->copy_ev[0], st));                       // after whatever the caller queued before
    STR_CUDA_OK(cudaStreamWaitEvent(ctx->copy_stream, ctx->copy_ev[0], 0));
    int nblk = 0;
    for (size_t r0 = 0; r0 < Rin; r0 += per, ++nblk) {
        const size_t nr = Rin - r0 < per ? Rin - r0 : per;
        STR_CUDA_OK(cudaMemcpyAsync((char *)in_dev + r0 * d->D * e, (const char *)hidden_in_host + r0 * d->D * e, nr * d->D * e,
                                    cudaMemcpyHostToDevice, ctx->copy_stream));
        STR_CUDA_OK(cudaEventRecord(ctx->copy_ev[1 + nblk], ctx->copy_stream));
    }
    const StackFeed feed = {nblk, (int)per, ctx->copy_ev + 1, OUT_CHUNKS, ctx->copy_ev + 9, ctx->copy_stream, hidden_out_host};
    int rc = stack_prefill_impl(ctx, d, nullptr, in_dev, out_dev, pos_dev, idx_dev, nullptr, nullptr, ws,
                                workspace_bytes - (size_t)(ws - (char *)workspace), stream, &feed);
    if (rc != STR_OK) return rc;
    // the hidden rows have gone out block by block on the copy stream; the caller's stream joins it before returning
    STR_CUDA_OK(cudaEventRecord(ctx->copy_ev[17], ctx->copy_stream));
    STR_CUDA_OK(cudaStreamWaitEvent(st, ctx->copy_ev[17], 0));
    if (idx_map_out_host)
        STR_CUDA_OK(cudaMemcpyAsync(idx_map_out_host, idx_dev, Rout * 4, cudaMemcpyDeviceToHost, st));
    STR_CUDA_OK(cudaStreamSynchronize(st));
    return STR_OK;
}
