// out[M,N] = a[M,K] * w[N,K]^T (+ residual), plain fp32 FFMA tiles.  Used for STR_F32 and as the
// generic path for shapes the tensor-core GEMM does not tile.
#include "dispatch.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, THREADS = 256;

template <typename T>
__global__ void __launch_bounds__(THREADS)
gemm_simt_kernel(int M, int N, int K, const T *__restrict__ a, const T *__restrict__ w,
                 const T *__restrict__ residual, T *__restrict__ out, const float *__restrict__ ss_in, int nt_in,
                 float inv_dim, float eps) {
    __shared__ float As[BK][BM + 1];
    __shared__ float Ws[BK][BN + 1];
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int e = tid; e < BM * BK; e += THREADS) {
            const int r = e / BK, c = e % BK;
            As[c][r] = (m0 + r < M && k0 + c < K) ? ldf(a + (size_t)(m0 + r) * K + k0 + c) : 0.f;
            Ws[c][r] = (n0 + r < N && k0 + c < K) ? ldf(w + (size_t)(n0 + r) * K + k0 + c) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float av[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[k][ty + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) wv[j] = Ws[k][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int mrow = m0 + ty + 16 * i;
        float scale = 1.0f;                       // fused RMSNorm of the A row (partials summed in index order)
        if (ss_in && mrow < M) {
            float t = 0.f;
            for (int j = 0; j < nt_in; ++j) t += ss_in[(size_t)mrow * nt_in + j];
            scale = rsqrtf(t * inv_dim + eps);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = mrow, n = n0 + tx + 16 * j;
            if (m < M && n < N) {
                float v = acc[i][j] * scale;
                if (residual) v += ldf(residual + (size_t)m * N + n);
                stf(out + (size_t)m * N + n, v);
            }
        }
    }
}

// Partial sums of squares of the stored rows, one partial per STR_SS_BLOCK columns.  One thread per (row, block)
// adds the squares in column order with fused multiply-adds: exactly the order in which the tensor-core GEMM's
// epilogue accumulates the same partial, so a hidden state gets bit-identical partials whether a GEMM epilogue or
// this kernel computed them (a stack is then exactly the composition of its layers run one by one).
template <typename T>
__global__ void __launch_bounds__(256)
row_sumsq_kernel(int rows, int D, int nt, const T *__restrict__ in, float *__restrict__ ss_out) {
    const long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= (long long)rows * nt) return;
    const int r = (int)(w / nt), j = (int)(w % nt);
    const int c0 = j * STR_SS_BLOCK, c1 = min(D, c0 + STR_SS_BLOCK);
    const T *p = in + (size_t)r * D;
    float ss = 0.f;
    for (int c = c0; c < c1; ++c) { const float v = ldf(p + c); ss = fmaf(v, v, ss); }
    ss_out[w] = ss;
}
template <>
__global__ void __launch_bounds__(256)
row_sumsq_kernel<__nv_bfloat16>(int rows, int D, int nt, const __nv_bfloat16 *__restrict__ in, float *__restrict__ ss_out) {
    const long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= (long long)rows * nt) return;
    const int r = (int)(w / nt), j = (int)(w % nt);
    const int c0 = j * STR_SS_BLOCK, c1 = min(D, c0 + STR_SS_BLOCK);
    const __nv_bfloat16 *p = in + (size_t)r * D;
    float ss = 0.f;
    int c = c0;
    if ((((uintptr_t)p) & 15) == 0 && (D & 7) == 0) {            // 16-byte loads, eight columns at a time, same column order
        for (; c + 8 <= c1; c += 8) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p + c));
            const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float lo = __uint_as_float(wv[q] << 16), hi = __uint_as_float(wv[q] & 0xFFFF0000u);
                ss = fmaf(lo, lo, ss);
                ss = fmaf(hi, hi, ss);
            }
        }
    }
    for (; c < c1; ++c) { const float v = __bfloat162float(p[c]); ss = fmaf(v, v, ss); }
    ss_out[w] = ss;
}

}  // namespace

int str_row_sumsq(str_ctx *ctx, int dtype, int rows, int D, const void *in, float *ss_out, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !in || !ss_out || rows < 0 || D <= 0) return STR_ERR_INVALID_ARG;
    if (rows == 0) return STR_OK;
    const int nt = str_ss_blocks(D);
    const int blocks = (int)(((long long)rows * nt + 255) / 256);
    if (dtype == STR_BF16)
        row_sumsq_kernel<__nv_bfloat16><<<blocks, 256, 0, (cudaStream_t)stream>>>(rows, D, nt, (const __nv_bfloat16 *)in, ss_out);
    else
        row_sumsq_kernel<float><<<blocks, 256, 0, (cudaStream_t)stream>>>(rows, D, nt, (const float *)in, ss_out);
    return str_launch_ok(ctx);
}

int str_gemm_simt(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
                  const void *residual, void *out, const StrRowNorm &rn, cudaStream_t st) {
    dim3 grid(ceil_div(N, BN), ceil_div(M, BM));
    if (dtype == STR_BF16)
        gemm_simt_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(M, N, K, (const __nv_bfloat16 *)a,
                                                                 (const __nv_bfloat16 *)w,
                                                                 (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)out,
                                                                 rn.ss_in, rn.nt_in, rn.inv_dim, rn.eps);
    else
        gemm_simt_kernel<float><<<grid, THREADS, 0, st>>>(M, N, K, (const float *)a, (const float *)w,
                                                         (const float *)residual, (float *)out, rn.ss_in, rn.nt_in,
                                                         rn.inv_dim, rn.eps);
    int rc = str_launch_ok(ctx);
    // the partial sums of squares of the stored output rows, by a second pass over what was just written
    if (rc == STR_OK && rn.ss_out) {
        const int nt = str_ss_blocks(N);
        const int blocks = (int)(((long long)M * nt + 255) / 256);
        if (dtype == STR_BF16)
            row_sumsq_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(M, N, nt, (const __nv_bfloat16 *)out, rn.ss_out);
        else
            row_sumsq_kernel<float><<<blocks, 256, 0, st>>>(M, N, nt, (const float *)out, rn.ss_out);
        rc = str_launch_ok(ctx);
    }
    return rc;
}
