// Attention importance normalised by the model's own causal row: the softmax denominator of text query m
// also holds the text keys m' <= m, so the score is the probability mass the query really puts on each
// visual token.  The two passes of the visual-only score stay as they are; between them this kernel folds
// the text keys into each row's (max, sum): one warp per (sequence, head, text query) walks the text keys the
// query may see, the lanes sharing each dot product, and merges the result with the visual keys' statistics.
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
    const T *kb = k + (((size_t)b * Tlen + n_vis) * Hkv + kv) * d;      // text key m' is row m' from here, stride Hkv * d
    const size_t kstride = (size_t)Hkv * d;
    // The lanes share each dot product (element c = lane, lane + 32, ...: coalesced rows), four keys at a time so
    // that their loads and reductions overlap; every lane then carries the same running (max, sum).
    constexpr int QR = 8;                                        // query elements kept in registers: d <= 256
    float qv[QR];
#pragma unroll
    for (int j = 0; j < QR; ++j) qv[j] = (lane + 32 * j < d) ? ldf(qr + lane + 32 * j) : 0.f;
    float mx = -FLT_MAX, sm = 0.f;
    for (int mp0 = 0; mp0 <= m; mp0 += 4) {                      // causal: text keys up to and including the query's own
        float part[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const T *kr = kb + (size_t)min(mp0 + u, m) * kstride;
            float a = 0.f;
#pragma unroll
            for (int j = 0; j < QR; ++j)
                if (lane + 32 * j < d) a = fmaf(qv[j], ldf(kr + lane + 32 * j), a);
            for (int c = lane + 32 * QR; c < d; c += 32) a = fmaf(ldf(qr + c), ldf(kr + c), a);
            part[u] = a;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int u = 0; u < 4; ++u) part[u] += __shfl_xor_sync(0xffffffffu, part[u], o);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (mp0 + u > m) break;
            const float l = part[u] * sc;
            const float nm = fmaxf(mx, l);
            sm = sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm)) + (LOG2 ? exp2f(l - nm) : expf(l - nm));
            mx = nm;
        }
    }
    if (lane == 0) {
        const float vm = st_max[warp], vs = LOG2 ? 1.0f / st_sum[warp] : st_sum[warp];
        const float nm = fmaxf(vm, mx);
        const float tot = vs * (LOG2 ? exp2f(vm - nm) : expf(vm - nm)) + sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm));
        st_max[warp] = nm;
        st_sum[warp] = LOG2 ? 1.0f / tot : tot;
    }
}

// Same result, text rows staged in shared memory: one CTA per (sequence, query head) holds the head's text
// queries and text keys as fp32 (rows padded by 4 floats); the CTAs of a head and their warps deal the queries
// out among them, a warp's lanes own the keys
// m' = lane, lane + 32, ... (conflict-free rows), then a warp reduction of (max, sum).
template <typename T, bool LOG2>
__global__ void __launch_bounds__(256)
attn_text_keys_stats_smem_kernel(int Tlen, int Hq, int Hkv, int d, int n_vis, int n_text, float scale, const T *__restrict__ q,
                                 const T *__restrict__ k, float *__restrict__ st_max, float *__restrict__ st_sum) {
    extern __shared__ __align__(16) float sh[];
    const int ld = (d + 3) / 4 * 4 + 4;                         // rows 16-byte aligned; 16-byte loads of 8 lanes hit 32 banks
    float *Qs = sh, *Ks = sh + (size_t)n_text * ld;
    const int h = blockIdx.x, b = blockIdx.y, kv = h / (Hq / Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float sc = LOG2 ? scale * 1.4426950408889634f : scale;
    {   // stage both tiles in 16-byte pieces, eight loads per thread in flight
        constexpr int PER = 16 / (int)sizeof(T);                  // elements per piece
        const bool vec = (d % PER) == 0 && ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k)) & 15) == 0;
        if (vec) {
            const int ppr = d / PER, total = 2 * n_text * ppr;    // pieces per row; queries first, then keys
            for (int e0 = threadIdx.x; e0 < total; e0 += 8 * blockDim.x) {
                uint4 t[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int e = e0 + u * blockDim.x;
                    if (e < total) {
                        const int isk = e >= n_text * ppr, ee = isk ? e - n_text * ppr : e, r = ee / ppr, c = (ee - r * ppr) * PER;
                        const T *src = isk ? k + (((size_t)b * Tlen + n_vis + r) * Hkv + kv) * d + c
                                           : q + (((size_t)b * Tlen + n_vis + r) * Hq + h) * d + c;
                        t[u] = __ldg(reinterpret_cast<const uint4 *>(src));
                    }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int e = e0 + u * blockDim.x;
                    if (e < total) {
                        const int isk = e >= n_text * ppr, ee = isk ? e - n_text * ppr : e, r = ee / ppr, c = (ee - r * ppr) * PER;
                        float *dst = (isk ? Ks : Qs) + r * ld + c;
                        const T *v = reinterpret_cast<const T *>(&t[u]);
#pragma unroll
                        for (int x = 0; x < PER; ++x) dst[x] = ldf(v + x);
                    }
                }
            }
        } else {
            for (int e = threadIdx.x; e < n_text * d; e += blockDim.x) {
                const int r = e / d, c = e - r * d;
                Qs[r * ld + c] = ldf(q + (((size_t)b * Tlen + n_vis + r) * Hq + h) * d + c);
                Ks[r * ld + c] = ldf(k + (((size_t)b * Tlen + n_vis + r) * Hkv + kv) * d + c);
            }
        }
    }
    __syncthreads();
    for (int m = (int)blockIdx.z * 8 + warp; m < n_text; m += 8 * (int)gridDim.z) {
        const float *qr = Qs + m * ld;
        float mx = -FLT_MAX, sm = 0.f;
        for (int mp = lane; mp <= m; mp += 32) {
            const float *kr = Ks + mp * ld;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            int c = 0;
            for (; c + 4 <= d; c += 4) {
                const float4 qa = *reinterpret_cast<const float4 *>(qr + c), ka = *reinterpret_cast<const float4 *>(kr + c);
                a0 = fmaf(qa.x, ka.x, a0); a1 = fmaf(qa.y, ka.y, a1);
                a2 = fmaf(qa.z, ka.z, a2); a3 = fmaf(qa.w, ka.w, a3);
            }
            for (; c < d; ++c) a0 = fmaf(qr[c], kr[c], a0);
            const float l = ((a0 + a1) + (a2 + a3)) * sc;
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
            const size_t r = ((size_t)b * Hq + h) * n_text + m;
            const float vm = st_max[r], vs = LOG2 ? 1.0f / st_sum[r] : st_sum[r];
            const float nm = fmaxf(vm, mx);
            const float tot = vs * (LOG2 ? exp2f(vm - nm) : expf(vm - nm)) + sm * (LOG2 ? exp2f(mx - nm) : expf(mx - nm));
            st_max[r] = nm;
            st_sum[r] = LOG2 ? 1.0f / tot : tot;
        }
    }
}

template <typename T, bool LOG2>
int launch_text_keys(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k, float scale,
                     float *st_max, float *st_sum, cudaStream_t st) {
    const size_t smem = 2 * (size_t)n_text * ((s->d + 3) / 4 * 4 + 4) * sizeof(float);
    const int zsplit = n_text >= 64 ? 4 : 1;                    // CTAs per head: the queries are dealt out among them
    if (smem <= (size_t)ctx->max_smem_optin) {
        if (smem > 48 * 1024)
            STR_CUDA_OK(cudaFuncSetAttribute(attn_text_keys_stats_smem_kernel<T, LOG2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             ctx->max_smem_optin));
        attn_text_keys_stats_smem_kernel<T, LOG2><<<dim3(s->Hq, s->Bz, zsplit), 256, smem, st>>>(s->T, s->Hq, s->Hkv, s->d, n_vis, n_text, scale,
                                                                                        (const T *)q, (const T *)k, st_max, st_sum);
    } else {
        const long long rows = (long long)s->Bz * s->Hq * n_text;
        attn_text_keys_stats_kernel<T, LOG2><<<(unsigned)((rows * 32 + 255) / 256), 256, 0, st>>>(
            s->T, s->Hq, s->Hkv, s->d, n_vis, n_text, (int)rows, scale, (const T *)q, (const T *)k, st_max, st_sum);
    }
    return str_launch_ok(ctx);
}

}  // namespace

// Folds the text keys m' <= m into the row statistics [Bz * Hq * n_text] left by the first pass.
int str_attn_text_keys_stats(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k,
                             float scale, bool log2_inv, float *st_max, float *st_sum, cudaStream_t st) {
    if (s->dtype == STR_BF16)
        return log2_inv ? launch_text_keys<__nv_bfloat16, true>(ctx, s, n_vis, n_text, q, k, scale, st_max, st_sum, st)
                        : launch_text_keys<__nv_bfloat16, false>(ctx, s, n_vis, n_text, q, k, scale, st_max, st_sum, st);
    return log2_inv ? launch_text_keys<float, true>(ctx, s, n_vis, n_text, q, k, scale, st_max, st_sum, st)
                    : launch_text_keys<float, false>(ctx, s, n_vis, n_text, q, k, scale, st_max, st_sum, st);
}
