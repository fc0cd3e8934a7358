// Causal GQA softmax attention forward, plain fp32 FFMA flash-style kernel (one pass over the keys
// with a running row maximum and sum).  Generic path / STR_F32.
#include <float.h>

#include "dispatch.cuh"

namespace {

constexpr int BR = 64, BC = 64, THREADS = 256;

template <typename T, int D16>
__global__ void __launch_bounds__(THREADS)
attn_fwd_simt_kernel(int Tq, int Tlen, int Hq, int Hkv, float scale, const int32_t *__restrict__ row_pos,
                     const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, T *__restrict__ o) {
    constexpr int d = 16 * D16, LDK = d + 1, LDP = BC + 1;
    extern __shared__ float smem[];
    float *Qs = smem;                // [BR][d+1]
    float *Ks = Qs + BR * LDK;       // [BC][d+1]
    float *Vs = Ks + BC * LDK;       // [BC][d]
    float *Ps = Vs + BC * d;         // [BR][BC+1]
    const int b = blockIdx.z, h = blockIdx.y, kv = h / (Hq / Hkv);
    const int r0 = (gridDim.x - 1 - blockIdx.x) * BR;     // longest rows first
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    // Query rows may be a gathered subset: row r then attends to the keys 0 .. row_pos[r] (ascending in r).
    const int32_t *rp = row_pos ? row_pos + (size_t)b * Tq : nullptr;
    auto key_index = [&](int r) -> int { r = min(r, Tq - 1); return rp ? min(max(rp[r], 0), Tlen - 1) : r; };
    const T *qb = q + ((size_t)b * Tq * Hq + h) * d;
    const T *kb = k + ((size_t)b * Tlen * Hkv + kv) * d;
    const T *vb = v + ((size_t)b * Tlen * Hkv + kv) * d;
    T *ob = o + ((size_t)b * Tq * Hq + h) * d;
    for (int e = tid; e < BR * d; e += THREADS) {
        const int r = e / d, c = e % d;
        Qs[r * LDK + c] = (r0 + r < Tq) ? ldf(qb + (size_t)(r0 + r) * Hq * d + c) * scale : 0.f;
    }
    int t_row[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) t_row[a] = key_index(r0 + ty + 16 * a);
    float mx[4], sm[4], acc[4][D16];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        mx[a] = -FLT_MAX;
        sm[a] = 0.f;
#pragma unroll
        for (int c = 0; c < D16; ++c) acc[a][c] = 0.f;
    }
    const int last_key = min(Tlen, key_index(r0 + BR - 1) + 1);
    for (int c0 = 0; c0 < last_key; c0 += BC) {
        __syncthreads();
        for (int e = tid; e < BC * d; e += THREADS) {
            const int r = e / d, c = e % d;
            const bool ok = c0 + r < Tlen;
            Ks[r * LDK + c] = ok ? ldf(kb + (size_t)(c0 + r) * Hkv * d + c) : 0.f;
            Vs[r * d + c] = ok ? ldf(vb + (size_t)(c0 + r) * Hkv * d + c) : 0.f;
        }
        __syncthreads();
        float s4[4][4] = {};
        for (int c = 0; c < d; ++c) {
            float qv[4], kvv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) qv[a] = Qs[(ty + 16 * a) * LDK + c];
#pragma unroll
            for (int j = 0; j < 4; ++j) kvv[j] = Ks[(tx + 16 * j) * LDK + c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int j = 0; j < 4; ++j) s4[a][j] = fmaf(qv[a], kvv[j], s4[a][j]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float tmax = -FLT_MAX;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = c0 + tx + 16 * j;
                if (key > t_row[a] || key >= Tlen) s4[a][j] = -FLT_MAX;
                tmax = fmaxf(tmax, s4[a][j]);
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
            const float nm = fmaxf(mx[a], tmax);
            const float corr = expf(mx[a] - nm);
            float psum = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float pv = s4[a][j] == -FLT_MAX ? 0.f : expf(s4[a][j] - nm);
                Ps[(ty + 16 * a) * LDP + tx + 16 * j] = pv;
                psum += pv;
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
            sm[a] = sm[a] * corr + psum;
            mx[a] = nm;
#pragma unroll
            for (int c = 0; c < D16; ++c) acc[a][c] *= corr;
        }
        __syncthreads();
        for (int j = 0; j < BC; ++j) {
            float pv[4], vv[D16];
#pragma unroll
            for (int a = 0; a < 4; ++a) pv[a] = Ps[(ty + 16 * a) * LDP + j];
#pragma unroll
            for (int c = 0; c < D16; ++c) vv[c] = Vs[j * d + tx + 16 * c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < D16; ++c) acc[a][c] = fmaf(pv[a], vv[c], acc[a][c]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int row = r0 + ty + 16 * a;
        if (row < Tq) {
            const float inv = 1.0f / sm[a];
#pragma unroll
            for (int c = 0; c < D16; ++c) stf(ob + (size_t)row * Hq * d + tx + 16 * c, acc[a][c] * inv);
        }
    }
}

template <typename T, int D16>
int launch(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos, const void *k, const void *v,
           float scale, void *o, cudaStream_t st) {
    constexpr int d = 16 * D16;
    const size_t smem = sizeof(float) * (size_t)(BR * (d + 1) + BC * (d + 1) + BC * d + BR * (BC + 1));
    STR_CUDA_OK(cudaFuncSetAttribute(attn_fwd_simt_kernel<T, D16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(ceil_div(n_rows, BR), s->Hq, s->Bz);
    attn_fwd_simt_kernel<T, D16><<<grid, THREADS, smem, st>>>(n_rows, s->T, s->Hq, s->Hkv, scale, row_pos, (const T *)q,
                                                              (const T *)k, (const T *)v, (T *)o);
    return str_launch_ok(ctx);
}

template <typename T>
int dispatch_d(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos, const void *k,
               const void *v, float scale, void *o, cudaStream_t st) {
    switch (s->d) {
        case 16: return launch<T, 1>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st);
        case 32: return launch<T, 2>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st);
        case 64: return launch<T, 4>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st);
        case 128: return launch<T, 8>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st);
        default: return STR_ERR_UNSUPPORTED_SHAPE;
    }
}

}  // namespace

int str_attn_prefill_simt(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos,
                          const void *k, const void *v, float scale, void *o, cudaStream_t st) {
    return s->dtype == STR_BF16 ? dispatch_d<__nv_bfloat16>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st)
                                : dispatch_d<float>(ctx, s, n_rows, q, row_pos, k, v, scale, o, st);
}
