// Attention importance normalised by the model's own causal row: the softmax denominator of text query m
// also holds the text keys m' <= m, so the score is the probability mass the query really puts on each
// visual token.  The two passes of the visual-only score stay as they are; between them this kernel folds
// the text keys into each row's (max, sum): one warp per (sequence, head, text query), lanes over the text
// keys, online max / sum per lane, warp reduction, then the merge with the visual keys' statistics.
#include <float.h>

#include "common.cuh"
#include "dispatch.cuh"

namespace {

// LOG2: statistics are kept as (max of logit * log2 e, 1 / sum) -- the tensor-core path; otherwise as
// (max of logit, sum) -- the plain path.
template <typename T, bool LOG2>
__global__ void __launch_bounds__(256)
attn_text_keys_stats_kernel(int Tlen, int Hq, int Hkv, int d, int n_vis, int n_text, int rows, float scale,
                            const T *__restrict__ q, const T *__restrict__ k, float *__restrict__ st_max,
                            float *__restrict__ st_sum) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= rows) return;                                    // r = (b * Hq + h) * n_text + m
    const int m = warp % n_text, bh = warp / n_text, h = bh % Hq, b = bh / Hq;
    const int kv = h / (Hq / Hkv);
    const float sc = LOG2 ? scale * 1.4426950408889634f : scale;
    const T *qr = q + (((size_t)b * Tlen + n_vis + m) * Hq + h) * d;
    float mx = -FLT_MAX, sm = 0.f;
    for (int mp = lane; mp <= m; mp += 32) {                     // causal: text keys up to and including the query's own
        const T *kr = k + (((size_t)b * Tlen + n_vis + mp) * Hkv + kv) * d;
        float a0 = 0.f, a1 = 0.f;
        int c = 0;
        for (; c + 2 <= d; c += 2) { a0 = fmaf(ldf(qr + c), ldf(kr + c), a0); a1 = fmaf(ldf(qr + c + 1), ldf(kr + c + 1), a1); }
        if (c < d) a0 = fmaf(ldf(qr + c), ldf(kr + c), a0);
        const float l = (a0 + a1) * sc;
        const float nm = fmaxf(mx, l);
        sm = sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm)) + (LOG2 ? exp2f(l - nm) : expf(l - nm));
        mx = nm;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sm, o);
        const float nm = fmaxf(mx, om);
        sm = sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm)) + os * (LOG2 ? exp2f(om - nm) : expf(om - nm));
        mx = nm;
    }
    if (lane == 0) {
        const float vm = st_max[warp], vs = LOG2 ? 1.0f / st_sum[warp] : st_sum[warp];
        const float nm = fmaxf(vm, mx);
        const float tot = vs * (LOG2 ? exp2f(vm - nm) : expf(vm - nm)) + sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm));
        st_max[warp] = nm;
        st_sum[warp] = LOG2 ? 1.0f / tot : tot;
    }
}

}  // namespace

// Folds the text keys m' <= m into the row statistics [Bz * Hq * n_text] left by the first pass.
int str_attn_text_keys_stats(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k,
                             float scale, bool log2_inv, float *st_max, float *st_sum, cudaStream_t st) {
    const long long rows = (long long)s->Bz * s->Hq * n_text;
    const unsigned blocks = (unsigned)((rows * 32 + 255) / 256);
#define STR_LAUNCH_TK(TT, L2)                                                                                                  \
    attn_text_keys_stats_kernel<TT, L2><<<blocks, 256, 0, st>>>(s->T, s->Hq, s->Hkv, s->d, n_vis, n_text, (int)rows, scale,    \
                                                                 (const TT *)q, (const TT *)k, st_max, st_sum)
    if (s->dtype == STR_BF16) {
        if (log2_inv) STR_LAUNCH_TK(__nv_bfloat16, true); else STR_LAUNCH_TK(__nv_bfloat16, false);
    } else {
        if (log2_inv) STR_LAUNCH_TK(float, true); else STR_LAUNCH_TK(float, false);
    }
#undef STR_LAUNCH_TK
    return str_launch_ok(ctx);
}
