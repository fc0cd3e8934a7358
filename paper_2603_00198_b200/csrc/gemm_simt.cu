// out[M,N] = a[M,K] * w[N,K]^T (+ residual), plain fp32 FFMA tiles.  Used for STR_F32 and as the
// generic path for shapes the tensor-core GEMM does not tile.
#include "dispatch.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, THREADS = 256;

template <typename T>
__global__ void __launch_bounds__(THREADS)
gemm_simt_kernel(int M, int N, int K, const T *__restrict__ a, const T *__restrict__ w,
                 const T *__restrict__ residual, T *__restrict__ out) {
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
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty + 16 * i, n = n0 + tx + 16 * j;
            if (m < M && n < N) {
                float v = acc[i][j];
                if (residual) v += ldf(residual + (size_t)m * N + n);
                stf(out + (size_t)m * N + n, v);
            }
        }
}

}  // namespace

int str_gemm_simt(str_ctx *ctx, int dtype, int M, int N, int K, const void *a, const void *w,
                  const void *residual, void *out, cudaStream_t st) {
    dim3 grid(ceil_div(N, BN), ceil_div(M, BM));
    if (dtype == STR_BF16)
        gemm_simt_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(M, N, K, (const __nv_bfloat16 *)a,
                                                                 (const __nv_bfloat16 *)w,
                                                                 (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)out);
    else
        gemm_simt_kernel<float><<<grid, THREADS, 0, st>>>(M, N, K, (const float *)a, (const float *)w,
                                                         (const float *)residual, (float *)out);
    return str_launch_ok(ctx);
}
