// Importance scores, plain fp32 FFMA kernels (used for STR_F32 inputs and as the generic path
// for shapes the tensor-core kernels do not tile).
//   Mamba (Eq. 2):   s_i = 1/(M G) sum_g dbar_i^g sum_m | b_i^g . c_m^g |
//   attention:       s_i = 1/(M Hq) sum_{m,h} softmax_i( q_m^h . k_i^kv(h) * scale )
// Delta-bar is a positive scalar per (token, group), so it is applied after the absolute value,
// in fp32, and never rounded into the operands.
#include <float.h>

#include "common.cuh"
#include <atomic>

#include "dispatch.cuh"

namespace {

constexpr int TI = 64;        // visual tokens (keys) per CTA tile
constexpr int TM = 16;        // text rows per inner block
constexpr int THREADS = 256;  // = TI * 4 row groups; each thread: 1 token x 4 text rows

// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(THREADS)
mamba_importance_kernel(int Tlen, int H, int n, int G, int n_vis, int n_text,
                        const T *__restrict__ B, const T *__restrict__ C, const float *__restrict__ dt,
                        float *__restrict__ scores) {
    extern __shared__ float smem[];
    const int ldk = n + 1;
    float *Bs = smem;                 // [TI][n+1]
    float *Cs = Bs + TI * ldk;        // [TM][n+1]
    float *red = Cs + TM * ldk;       // [4][TI]
    const int b = blockIdx.y, i0 = blockIdx.x * TI;
    const int tid = threadIdx.x, ti = tid % TI, rg = tid / TI;
    const int hpg = H / G;
    const T *Bb = B + (size_t)b * Tlen * G * n;
    const T *Cb = C + (size_t)b * Tlen * G * n;
    const float *dtb = dt + (size_t)b * Tlen * H;
    const int i = i0 + ti;
    float total = 0.f;
    for (int g = 0; g < G; ++g) {
        __syncthreads();
        for (int e = tid; e < TI * n; e += THREADS) {
            const int r = e / n, c = e % n;
            Bs[r * ldk + c] = (i0 + r < n_vis) ? ldf(Bb + ((size_t)(i0 + r) * G + g) * n + c) : 0.f;
        }
        float acc = 0.f;
        for (int m0 = 0; m0 < n_text; m0 += TM) {
            __syncthreads();
            for (int e = tid; e < TM * n; e += THREADS) {
                const int r = e / n, c = e % n;
                Cs[r * ldk + c] = (m0 + r < n_text) ? ldf(Cb + ((size_t)(n_vis + m0 + r) * G + g) * n + c) : 0.f;
            }
            __syncthreads();
            float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
            const float *bp = Bs + ti * ldk;
            const float *cp = Cs + (rg * 4) * ldk;
            for (int c = 0; c < n; ++c) {
                const float bv = bp[c];
                d0 = fmaf(bv, cp[c], d0);
                d1 = fmaf(bv, cp[ldk + c], d1);
                d2 = fmaf(bv, cp[2 * ldk + c], d2);
                d3 = fmaf(bv, cp[3 * ldk + c], d3);
            }
            acc += fabsf(d0) + fabsf(d1) + fabsf(d2) + fabsf(d3);   // padded rows are zero
        }
        float dbar = 0.f;
        if (i < n_vis) {
            for (int h = 0; h < hpg; ++h) dbar += dtb[(size_t)i * H + g * hpg + h];
            dbar /= (float)hpg;
        }
        total = fmaf(dbar, acc, total);
    }
    red[rg * TI + ti] = total;
    __syncthreads();
    if (rg == 0 && i < n_vis)
        scores[(size_t)b * n_vis + i] =
            (red[ti] + red[TI + ti] + red[2 * TI + ti] + red[3 * TI + ti]) / ((float)n_text * (float)G);
}

// ------------------------------------------------------------------------------------------
// Attention pass 1: row maximum and sum of exp over the visual keys for TM query rows of one head.
template <typename T>
__global__ void __launch_bounds__(THREADS)
attn_rowstats_kernel(int Tlen, int Hq, int Hkv, int d, int n_vis, int n_text, float scale,
                     const T *__restrict__ q, const T *__restrict__ k,
                     float *__restrict__ row_max, float *__restrict__ row_sum) {
    extern __shared__ float smem[];
    const int ldk = d + 1;
    float *Ks = smem;                  // [TI][d+1]
    float *Qs = Ks + TI * ldk;         // [TM][d+1]
    float *red_m = Qs + TM * ldk;      // [TM][TI]
    float *red_s = red_m + TM * TI;    // [TM][TI]
    const int b = blockIdx.z, h = blockIdx.y, m0 = blockIdx.x * TM;
    const int kv = h / (Hq / Hkv);
    const int tid = threadIdx.x, ti = tid % TI, rg = tid / TI;
    const T *qb = q + (size_t)b * Tlen * Hq * d;
    const T *kb = k + (size_t)b * Tlen * Hkv * d;
    for (int e = tid; e < TM * d; e += THREADS) {
        const int r = e / d, c = e % d;
        Qs[r * ldk + c] = (m0 + r < n_text) ? ldf(qb + ((size_t)(n_vis + m0 + r) * Hq + h) * d + c) : 0.f;
    }
    float mx[4], sm[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { mx[j] = -FLT_MAX; sm[j] = 0.f; }
    for (int i0 = 0; i0 < n_vis; i0 += TI) {
        __syncthreads();
        for (int e = tid; e < TI * d; e += THREADS) {
            const int r = e / d, c = e % d;
            Ks[r * ldk + c] = (i0 + r < n_vis) ? ldf(kb + ((size_t)(i0 + r) * Hkv + kv) * d + c) : 0.f;
        }
        __syncthreads();
        float d4[4] = {0.f, 0.f, 0.f, 0.f};
        const float *kp = Ks + ti * ldk;
        const float *qp = Qs + (rg * 4) * ldk;
        for (int c = 0; c < d; ++c) {
            const float kvv = kp[c];
#pragma unroll
            for (int j = 0; j < 4; ++j) d4[j] = fmaf(kvv, qp[j * ldk + c], d4[j]);
        }
        if (i0 + ti < n_vis) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float l = d4[j] * scale;
                const float nm = fmaxf(mx[j], l);
                sm[j] = sm[j] * expf(mx[j] - nm) + expf(l - nm);
                mx[j] = nm;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) { red_m[(rg * 4 + j) * TI + ti] = mx[j]; red_s[(rg * 4 + j) * TI + ti] = sm[j]; }
    __syncthreads();
    if (tid < TM && m0 + tid < n_text) {
        float M_ = -FLT_MAX;
        for (int t = 0; t < TI; ++t) M_ = fmaxf(M_, red_m[tid * TI + t]);
        float S_ = 0.f;
        for (int t = 0; t < TI; ++t) S_ += red_s[tid * TI + t] * expf(red_m[tid * TI + t] - M_);
        const size_t o = ((size_t)b * Hq + h) * n_text + m0 + tid;
        row_max[o] = M_;
        row_sum[o] = S_;
    }
}

// Attention pass 2: for a tile of TI keys, sum over all heads and text rows of
// exp(logit - row_max) / row_sum.  Deterministic: one CTA owns a key tile, no atomics.
template <typename T>
__global__ void __launch_bounds__(THREADS)
attn_colsum_kernel(int Tlen, int Hq, int Hkv, int d, int n_vis, int n_text, float scale,
                   const T *__restrict__ q, const T *__restrict__ k,
                   const float *__restrict__ row_max, const float *__restrict__ row_sum,
                   float *__restrict__ scores) {
    extern __shared__ float smem[];
    const int ldk = d + 1;
    float *Ks = smem;                  // [TI][d+1]
    float *Qs = Ks + TI * ldk;         // [TM][d+1]
    float *stat = Qs + TM * ldk;       // [2][TM]
    float *red = stat + 2 * TM;        // [4][TI]
    const int b = blockIdx.y, i0 = blockIdx.x * TI;
    const int tid = threadIdx.x, ti = tid % TI, rg = tid / TI;
    const int qpk = Hq / Hkv;
    const T *qb = q + (size_t)b * Tlen * Hq * d;
    const T *kb = k + (size_t)b * Tlen * Hkv * d;
    float total = 0.f;
    for (int kv = 0; kv < Hkv; ++kv) {
        __syncthreads();
        for (int e = tid; e < TI * d; e += THREADS) {
            const int r = e / d, c = e % d;
            Ks[r * ldk + c] = (i0 + r < n_vis) ? ldf(kb + ((size_t)(i0 + r) * Hkv + kv) * d + c) : 0.f;
        }
        for (int hh = 0; hh < qpk; ++hh) {
            const int h = kv * qpk + hh;
            for (int m0 = 0; m0 < n_text; m0 += TM) {
                __syncthreads();
                for (int e = tid; e < TM * d; e += THREADS) {
                    const int r = e / d, c = e % d;
                    Qs[r * ldk + c] = (m0 + r < n_text) ? ldf(qb + ((size_t)(n_vis + m0 + r) * Hq + h) * d + c) : 0.f;
                }
                if (tid < TM) {
                    const bool ok = m0 + tid < n_text;
                    const size_t o = ((size_t)b * Hq + h) * n_text + m0 + tid;
                    stat[tid] = ok ? row_max[o] : 0.f;
                    stat[TM + tid] = ok ? 1.0f / row_sum[o] : 0.f;    // padded rows contribute 0
                }
                __syncthreads();
                float d4[4] = {0.f, 0.f, 0.f, 0.f};
                const float *kp = Ks + ti * ldk;
                const float *qp = Qs + (rg * 4) * ldk;
                for (int c = 0; c < d; ++c) {
                    const float kvv = kp[c];
#pragma unroll
                    for (int j = 0; j < 4; ++j) d4[j] = fmaf(kvv, qp[j * ldk + c], d4[j]);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    total += expf(d4[j] * scale - stat[rg * 4 + j]) * stat[TM + rg * 4 + j];
            }
        }
    }
    __syncthreads();
    red[rg * TI + ti] = total;
    __syncthreads();
    if (rg == 0 && i0 + ti < n_vis)
        scores[(size_t)b * n_vis + i0 + ti] =
            (red[ti] + red[TI + ti] + red[2 * TI + ti] + red[3 * TI + ti]) / ((float)n_text * (float)Hq);
}

template <typename T>
int launch_mamba_importance(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B,
                            const void *C, const float *dt, float *scores, cudaStream_t st) {
    const size_t smem = ((size_t)(TI + TM) * (s->n + 1) + 4 * TI) * sizeof(float);
    if (smem > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    STR_CUDA_OK(cudaFuncSetAttribute(mamba_importance_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(ceil_div(n_vis, TI), s->Bz);
    mamba_importance_kernel<T><<<grid, THREADS, smem, st>>>(s->T, s->H, s->n, s->G, n_vis, n_text, (const T *)B,
                                                           (const T *)C, dt, scores);
    return str_launch_ok(ctx);
}

template <typename T>
int launch_attn_importance(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q,
                           const void *k, float scale, float *scores, float *row_max, float *row_sum,
                           bool causal_row, cudaStream_t st) {
    const size_t smem1 = ((size_t)(TI + TM) * (s->d + 1) + 2 * TM * TI) * sizeof(float);
    const size_t smem2 = ((size_t)(TI + TM) * (s->d + 1) + 2 * TM + 4 * TI) * sizeof(float);
    if (smem1 > (size_t)ctx->max_smem_optin || smem2 > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    STR_CUDA_OK(cudaFuncSetAttribute(attn_rowstats_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1));
    STR_CUDA_OK(cudaFuncSetAttribute(attn_colsum_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
    dim3 g1(ceil_div(n_text, TM), s->Hq, s->Bz);
    attn_rowstats_kernel<T><<<g1, THREADS, smem1, st>>>(s->T, s->Hq, s->Hkv, s->d, n_vis, n_text, scale, (const T *)q,
                                                        (const T *)k, row_max, row_sum);
    int rc = str_launch_ok(ctx);
    if (rc == STR_OK && causal_row)
        rc = str_attn_text_keys_stats(ctx, s, n_vis, n_text, q, k, scale, false, row_max, row_sum, st);
    if (rc != STR_OK) return rc;
    dim3 g2(ceil_div(n_vis, TI), s->Bz);
    attn_colsum_kernel<T><<<g2, THREADS, smem2, st>>>(s->T, s->Hq, s->Hkv, s->d, n_vis, n_text, scale, (const T *)q,
                                                      (const T *)k, row_max, row_sum, scores);
    return str_launch_ok(ctx);
}

}  // namespace

int str_mamba_importance_simt(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B,
                              const void *C, const float *dt, float *scores, cudaStream_t st) {
    return s->dtype == STR_BF16
               ? launch_mamba_importance<__nv_bfloat16>(ctx, s, n_vis, n_text, B, C, dt, scores, st)
               : launch_mamba_importance<float>(ctx, s, n_vis, n_text, B, C, dt, scores, st);
}

int str_attn_importance_simt(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q,
                             const void *k, float scale, float *scores, float *row_max, float *row_sum,
                             bool causal_row, cudaStream_t st) {
    return s->dtype == STR_BF16
               ? launch_attn_importance<__nv_bfloat16>(ctx, s, n_vis, n_text, q, k, scale, scores, row_max, row_sum, causal_row, st)
               : launch_attn_importance<float>(ctx, s, n_vis, n_text, q, k, scale, scores, row_max, row_sum, causal_row, st);
}

// ------------------------------------------------------------------------------------------
// Allocation-free attention importance.  Some callers may not allocate device memory at all: a
// plug-in running inside a host whose memory pool is fixed at start-up, a real-time loop that must
// not hit the allocator's lock, or code that is handed raw pointers and owns no allocator.  For them
// the row statistics of the first pass live in a fixed array inside the library image instead of a
// caller workspace.  Every GPU that loads the library carries the array until the process exits.
static __device__ __align__(256) float g_attn_static_rowstats[2 * STR_ATTN_STATIC_MAX_ROWS];

namespace {
constexpr int kMaxDevices = 64;
// device address of the array, per device (host cache; contexts on several host threads may race to fill an entry,
// and every one of them stores the same value)
std::atomic<float *> g_rowstats_dev_ptr[kMaxDevices];
}  // namespace

extern "C" int str_attn_importance_static(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text,
                                          const void *q, const void *k, float softmax_scale, float *scores_out,
                                          void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ATTN_SCORE, stream);
    if (!ctx || !s || !q || !k) return STR_ERR_INVALID_ARG;
    if (s->Bz <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Hq % s->Hkv != 0 || s->d <= 0 || n_vis < 0 || n_text <= 0 ||
        n_vis + n_text != s->T || (s->dtype != STR_F32 && s->dtype != STR_BF16))
        return STR_ERR_INVALID_ARG;
    const long long rows = (long long)s->Bz * s->Hq * n_text;
    if (rows > STR_ATTN_STATIC_MAX_ROWS) return STR_ERR_WORKSPACE_TOO_SMALL;   // beyond the built-in scratch
    if (n_vis == 0) return STR_OK;
    if (!scores_out) return STR_ERR_INVALID_ARG;
    if (ctx->device < 0 || ctx->device >= kMaxDevices) return STR_ERR_INVALID_ARG;
    float *base = g_rowstats_dev_ptr[ctx->device].load(std::memory_order_acquire);
    if (!base) {
        // One-time set-up per device: in host code the array's name is only a stand-in, so ask the
        // runtime for its device address, with the context's device current.
        int prev = -1;
        STR_CUDA_OK(cudaGetDevice(&prev));
        if (prev != ctx->device) STR_CUDA_OK(cudaSetDevice(ctx->device));
        void *sym = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&sym, g_attn_static_rowstats);
        if (prev != ctx->device) cudaSetDevice(prev);
        if (e != cudaSuccess || !sym) {
            (void)cudaGetLastError();             // do not leave the runtime's sticky error for an unrelated later call
            return STR_ERR_CUDA;
        }
        base = (float *)sym;
        g_rowstats_dev_ptr[ctx->device].store(base, std::memory_order_release);
    }
    // Both halves are fully rewritten by the first pass before the second pass reads them, so nothing
    // left over from an earlier call is ever used and nothing needs clearing.
    float *row_max = base, *row_sum = base + rows;
    return str_attn_importance_simt(ctx, s, n_vis, n_text, q, k, softmax_scale, scores_out, row_max, row_sum, false,
                                    (cudaStream_t)stream);
}
