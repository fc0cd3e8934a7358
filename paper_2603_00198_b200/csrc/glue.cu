// Element-wise / row-wise block glue around the mixers: RMSNorm, the Mamba-2 pre-scan step
// (causal depthwise conv + SiLU + split + softplus), gated RMSNorm, and RoPE + q/k/v split.
// All HBM-bound; each activation is read once and written once.
#include "dispatch.cuh"

namespace {

__device__ __forceinline__ float block_sum(float v, float *red) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    const int nw = (blockDim.x + 31) >> 5;
    for (int w = 0; w < nw; ++w) t += red[w];
    return t;
}

template <typename T>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(int D, float eps, const T *__restrict__ in, T *__restrict__ out) {
    __shared__ float red[32];
    const T *r = in + (size_t)blockIdx.x * D;
    T *o = out + (size_t)blockIdx.x * D;
    float ss = 0.f;
    for (int c = threadIdx.x; c < D; c += blockDim.x) { const float v = ldf(r + c); ss = fmaf(v, v, ss); }
    const float inv = rsqrtf(block_sum(ss, red) / (float)D + eps);
    for (int c = threadIdx.x; c < D; c += blockDim.x) stf(o + c, ldf(r + c) * inv);
}

// Source row of output row r when the rows are gathered on the fly (the same map as str_compact: per
// sequence the k kept visual rows, then the text rows); the identity when kept == nullptr.
// z_direct: the gate rows are already compacted (row r of z belongs to output row r); y is still gathered.
struct RowGather { const int32_t *kept; int T_in, n_vis, k, T_out; bool z_direct; };
__device__ __forceinline__ size_t gather_src_row(const RowGather &g, size_t r) {
    if (!g.kept) return r;
    const size_t b = r / g.T_out;
    const int j = (int)(r - b * g.T_out);
    const int src = j < g.k ? __ldg(g.kept + b * g.k + j) : g.n_vis + (j - g.k);
    return b * g.T_in + src;
}

template <typename T>
__global__ void __launch_bounds__(256)
gated_rmsnorm_kernel(int d_inner, int ld_z, float eps, const T *__restrict__ y, const T *__restrict__ z,
                     T *__restrict__ out, RowGather rg) {
    __shared__ float red[32];
    const size_t srow = gather_src_row(rg, blockIdx.x);
    const T *yr = y + srow * d_inner;
    const T *zr = z + (rg.z_direct ? (size_t)blockIdx.x : srow) * ld_z;
    T *o = out + (size_t)blockIdx.x * d_inner;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d_inner; c += blockDim.x) {
        const float v = ldf(yr + c) * silu_f(ldf(zr + c));
        ss = fmaf(v, v, ss);
    }
    const float inv = rsqrtf(block_sum(ss, red) / (float)d_inner + eps);
    for (int c = threadIdx.x; c < d_inner; c += blockDim.x)
        stf(o + c, ldf(yr + c) * silu_f(ldf(zr + c)) * inv);
}

// One thread per (token, conv channel); consecutive threads walk consecutive channels.
template <typename T>
__global__ void __launch_bounds__(256)
mamba_conv_split_kernel(int Tlen, int H, int p, int n, int G, int W, int zoff, const T *__restrict__ zxbcdt,
                        const float *__restrict__ conv_w, const float *__restrict__ conv_b,
                        const float *__restrict__ dt_bias, T *__restrict__ x_out, T *__restrict__ B_out,
                        T *__restrict__ C_out, float *__restrict__ dt_out) {
    const int d_inner = H * p, gn = G * n;
    const int conv_dim = d_inner + 2 * gn;
    const int ld = zoff + conv_dim + H;                  // zoff = d_inner with the z columns in front, 0 without
    const int cols = conv_dim + H;                       // conv channels, then the H dt columns
    const size_t row = blockIdx.x;                       // b * Tlen + t (grid.x: no 65535 limit)
    const int t = (int)(row % Tlen);
    const int c = blockIdx.y * blockDim.x + threadIdx.x;
    if (c >= cols) return;
    const T *base = zxbcdt + row * ld;
    if (c >= conv_dim) {
        const int h = c - conv_dim;
        dt_out[row * H + h] = softplus_f(ldf(base + zoff + conv_dim + h) + dt_bias[h]);
        return;
    }
    float acc = conv_b[c];
    for (int j = 0; j < W; ++j) {
        const int back = W - 1 - j;                      // tap j reads token t - (W-1) + j
        if (t - back >= 0) acc = fmaf(conv_w[(size_t)c * W + j], ldf(base - (size_t)back * ld + zoff + c), acc);
    }
    const float v = silu_f(acc);
    if (c < d_inner) stf(x_out + row * d_inner + c, v);
    else if (c < d_inner + gn) stf(B_out + row * gn + (c - d_inner), v);
    else stf(C_out + row * gn + (c - d_inner - gn), v);
}

// One thread per (token, head, pair index i < d/2) for q and k; v columns are copied.
template <typename T>
__global__ void __launch_bounds__(256)
rope_split_kernel(int Hq, int Hkv, int d, double log2_theta, const int32_t *__restrict__ positions,
                  const T *__restrict__ qkv, T *__restrict__ q_out, T *__restrict__ k_out, T *__restrict__ v_out) {
    const int half = d / 2;
    const int ld = (Hq + 2 * Hkv) * d;
    const size_t row = blockIdx.x;                       // grid.x: no 65535 limit
    const int e = blockIdx.y * blockDim.x + threadIdx.x;
    const int n_rot = (Hq + Hkv) * half;
    const int n_v = Hkv * d;
    const T *base = qkv + row * ld;
    if (e < n_rot) {
        const int head = e / half, i = e % half;
        // angle in fp64, reduced to [0, 2pi) before the fp32 sincos: positions reach tens of thousands
        const double inv_freq = exp2(-2.0 * (double)i / (double)d * log2_theta);
        double ang = (double)positions[row] * inv_freq;
        ang -= 6.283185307179586476925 * floor(ang * 0.15915494309189533576888);
        float sn, cs;
        sincosf((float)ang, &sn, &cs);
        const float a = ldf(base + head * d + i), b = ldf(base + head * d + half + i);
        T *dst = head < Hq ? q_out + (row * Hq + head) * d : k_out + (row * Hkv + (head - Hq)) * d;
        stf(dst + i, a * cs - b * sn);
        stf(dst + half + i, b * cs + a * sn);
    } else if (e < n_rot + n_v) {
        const int c = e - n_rot;
        v_out[row * n_v + c] = base[(Hq + Hkv) * d + c];
    }
}


// ---- 16-byte vectorised bf16 versions (used when the row length and strides are multiples of 8) ----
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[2 * j] = __uint_as_float(w[j] << 16);
        f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
    }
}
// SiLU for results that are stored as bf16: exp2 and reciprocal on the special-function unit (relative
// error about 2^-21, far below the 2^-9 of the storage rounding) instead of the exact exp and division.
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
    return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
}

// RMSNorm, one warp per row, the row held in registers between the reduction and the scaling
// (rows of up to 32 * 8 * VPL elements): each element is read once and written once.
template <int VPL>
__global__ void __launch_bounds__(256)
rmsnorm_bf16_vec_kernel(int rows, int D, float eps, const __nv_bfloat16 *__restrict__ in, __nv_bfloat16 *__restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int nvec = D >> 3;
    const uint4 *r = reinterpret_cast<const uint4 *>(in + (size_t)row * D);
    uint4 *o = reinterpret_cast<uint4 *>(out + (size_t)row * D);
    uint4 v[VPL];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int c = lane + 32 * i;
        v[i] = c < nvec ? __ldg(r + c) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        float f[8];
        unpack8(v[i], f);
#pragma unroll
        for (int j = 0; j < 8; ++j) ss = fmaf(f[j], f[j], ss);
    }
    const float inv = rsqrtf(warp_sum(ss) / (float)D + eps);
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int c = lane + 32 * i;
        if (c < nvec) {
            float f[8];
            unpack8(v[i], f);
#pragma unroll
            for (int j = 0; j < 8; ++j) f[j] *= inv;
            o[c] = pack8(f);
        }
    }
}

// Gated RMSNorm, one CTA per row, y * SiLU(z) held in registers (rows of up to 256 * 8 * VPT elements).
template <int VPT>
__global__ void __launch_bounds__(256)
gated_rmsnorm_bf16_vec_kernel(int d_inner, int ld_z, float eps, const __nv_bfloat16 *__restrict__ y,
                              const __nv_bfloat16 *__restrict__ z, __nv_bfloat16 *__restrict__ out, RowGather rg) {
    __shared__ float red[32];
    const int nvec = d_inner >> 3;
    const size_t srow = gather_src_row(rg, blockIdx.x);
    const uint4 *yr = reinterpret_cast<const uint4 *>(y + srow * d_inner);
    const uint4 *zr = reinterpret_cast<const uint4 *>(z + (rg.z_direct ? (size_t)blockIdx.x : srow) * ld_z);
    uint4 *o = reinterpret_cast<uint4 *>(out + (size_t)blockIdx.x * d_inner);
    uint4 yv[VPT], zv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int c = threadIdx.x + 256 * i;
        yv[i] = c < nvec ? __ldg(yr + c) : make_uint4(0u, 0u, 0u, 0u);
        zv[i] = c < nvec ? __ldg(zr + c) : make_uint4(0u, 0u, 0u, 0u);
    }
    float g[VPT][8];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        float fy[8], fz[8];
        unpack8(yv[i], fy);
        unpack8(zv[i], fz);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            g[i][j] = fy[j] * silu_fast(fz[j]);
            ss = fmaf(g[i][j], g[i][j], ss);
        }
    }
    const float inv = rsqrtf(block_sum(ss, red) / (float)d_inner + eps);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int c = threadIdx.x + 256 * i;
        if (c < nvec) {
#pragma unroll
            for (int j = 0; j < 8; ++j) g[i][j] *= inv;
            o[c] = pack8(g[i]);
        }
    }
}

// Mamba-2 pre-scan step, width-4 conv: one thread owns 4 consecutive conv channels and walks CONV_TT
// consecutive tokens with the three previous inputs held in registers, so every input element is
// read once (plus a 3-token halo per tile) and every output written once, as 8-byte vectors (a warp
// covers 256 contiguous bytes of a row).  Eight loads are in flight per thread and three CTAs fit an
// SM, which is what it takes to keep HBM busy from a kernel this short.  The last block row handles the
// dt columns.
constexpr int CONV_TT = 32, CONV_CPT = 4, CONV_UNROLL = 8;
__device__ __forceinline__ void unpack4(const uint2 &v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
}
__global__ void __launch_bounds__(256, 3)
mamba_conv_split_bf16_vec_kernel(int Tlen, int H, int p, int n, int G, int zoff, const __nv_bfloat16 *__restrict__ zxbcdt,
                                 const float *__restrict__ conv_w, const float *__restrict__ conv_b,
                                 const float *__restrict__ dt_bias, __nv_bfloat16 *__restrict__ x_out,
                                 __nv_bfloat16 *__restrict__ B_out, __nv_bfloat16 *__restrict__ C_out,
                                 float *__restrict__ dt_out) {
    const int d_inner = H * p, gn = G * n;
    const int conv_dim = d_inner + 2 * gn;
    const int ld = zoff + conv_dim + H;
    const int tiles = (Tlen + CONV_TT - 1) / CONV_TT;
    const int b = blockIdx.x / tiles, t0 = (blockIdx.x % tiles) * CONV_TT;
    const int t1 = min(Tlen, t0 + CONV_TT);
    const size_t row0 = (size_t)b * Tlen;
    if (blockIdx.y == gridDim.y - 1) {
        for (int e = threadIdx.x; e < (t1 - t0) * H; e += blockDim.x) {
            const int t = t0 + e / H, h = e % H;
            dt_out[(row0 + t) * H + h] =
                softplus_f(__bfloat162float(zxbcdt[(row0 + t) * ld + zoff + conv_dim + h]) + dt_bias[h]);
        }
        return;
    }
    const int c0 = (blockIdx.y * blockDim.x + threadIdx.x) * CONV_CPT;
    if (c0 >= conv_dim) return;
    float w[CONV_CPT][4], bias[CONV_CPT];
#pragma unroll
    for (int j = 0; j < CONV_CPT; ++j) {
        const float4 wv = __ldg(reinterpret_cast<const float4 *>(conv_w) + c0 + j);
        w[j][0] = wv.x; w[j][1] = wv.y; w[j][2] = wv.z; w[j][3] = wv.w;
        bias[j] = __ldg(conv_b + c0 + j);
    }
    __nv_bfloat16 *dst;
    int dst_ld;
    if (c0 < d_inner) { dst = x_out + c0; dst_ld = d_inner; }
    else if (c0 < d_inner + gn) { dst = B_out + (c0 - d_inner); dst_ld = gn; }
    else { dst = C_out + (c0 - d_inner - gn); dst_ld = gn; }
    const __nv_bfloat16 *src = zxbcdt + zoff + c0;
    float h3[CONV_CPT], h2[CONV_CPT], h1[CONV_CPT];     // inputs of tokens t-3, t-2, t-1
    {
        const uint2 zero = make_uint2(0u, 0u);
        unpack4(t0 >= 3 ? __ldg(reinterpret_cast<const uint2 *>(src + (row0 + t0 - 3) * ld)) : zero, h3);
        unpack4(t0 >= 2 ? __ldg(reinterpret_cast<const uint2 *>(src + (row0 + t0 - 2) * ld)) : zero, h2);
        unpack4(t0 >= 1 ? __ldg(reinterpret_cast<const uint2 *>(src + (row0 + t0 - 1) * ld)) : zero, h1);
    }
#pragma unroll 1
    for (int tb = t0; tb < t1; tb += CONV_UNROLL) {
        uint2 raw[CONV_UNROLL];
#pragma unroll
        for (int u = 0; u < CONV_UNROLL; ++u)
            raw[u] = (tb + u < t1) ? __ldg(reinterpret_cast<const uint2 *>(src + (row0 + tb + u) * ld)) : make_uint2(0u, 0u);
#pragma unroll
        for (int u = 0; u < CONV_UNROLL; ++u) {
            float cur[CONV_CPT], o[CONV_CPT];
            unpack4(raw[u], cur);
#pragma unroll
            for (int j = 0; j < CONV_CPT; ++j) {
                float acc = bias[j];
                acc = fmaf(w[j][0], h3[j], acc);
                acc = fmaf(w[j][1], h2[j], acc);
                acc = fmaf(w[j][2], h1[j], acc);
                acc = fmaf(w[j][3], cur[j], acc);
                o[j] = silu_fast(acc);
                h3[j] = h2[j]; h2[j] = h1[j]; h1[j] = cur[j];
            }
            if (tb + u < t1)
                *reinterpret_cast<uint2 *>(dst + (row0 + tb + u) * dst_ld) = make_uint2(pack2(o[0], o[1]), pack2(o[2], o[3]));
        }
    }
}

// The rows a fused in-projection epilogue (StrConvEpilogue) leaves out: rows r with r % 32 < 3, whose earlier rows
// sit in another warp of that epilogue.  The projection of rows r-3 .. r is in `zxbcdt` (the epilogue stores it for
// the first and the last three rows of every 32).  One thread: 8 channels (taps and bias held in registers) of
// EDGE_GROUPS consecutive 32-row groups, the arithmetic of mamba_conv_split_bf16_vec_kernel.
constexpr int EDGE_GROUPS = 8;
__global__ void __launch_bounds__(256)
mamba_conv_edge_rows_kernel(int rows, int Tlen, int ld, int zoff, int d_inner, int gn, const __nv_bfloat16 *__restrict__ zxbcdt,
                            const float *__restrict__ conv_w, const float *__restrict__ conv_b,
                            __nv_bfloat16 *__restrict__ x_out, __nv_bfloat16 *__restrict__ B_out,
                            __nv_bfloat16 *__restrict__ C_out) {
    const int c0 = (blockIdx.y * blockDim.x + threadIdx.x) * 8;
    if (c0 >= d_inner + 2 * gn) return;
    float4 w[8];
    float bias[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        w[j] = __ldg(reinterpret_cast<const float4 *>(conv_w) + c0 + j);
        bias[j] = __ldg(conv_b + c0 + j);
    }
    __nv_bfloat16 *dst;
    int dst_ld;
    if (c0 < d_inner) { dst = x_out + c0; dst_ld = d_inner; }
    else if (c0 < d_inner + gn) { dst = B_out + (c0 - d_inner); dst_ld = gn; }
    else { dst = C_out + (c0 - d_inner - gn); dst_ld = gn; }
    const __nv_bfloat16 *src = zxbcdt + zoff + c0;
    const int groups = (rows + 31) / 32;
#pragma unroll 2
    for (int gi = 0; gi < EDGE_GROUPS; ++gi) {
        const int grp = blockIdx.x * EDGE_GROUPS + gi;
        if (grp >= groups) break;
        const int r0 = grp * 32;
        uint4 raw[6];
#pragma unroll
        for (int i = 0; i < 6; ++i) {
            const int r = r0 - 3 + i;
            raw[i] = (r >= 0 && r < rows) ? __ldg(reinterpret_cast<const uint4 *>(src + (size_t)r * ld)) : make_uint4(0u, 0u, 0u, 0u);
        }
        float h[6][8];
#pragma unroll
        for (int i = 0; i < 6; ++i) unpack8(raw[i], h[i]);
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const int r = r0 + k;
            if (r < rows) {
                const int t_in = r % Tlen;
                float o[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float acc = bias[j];
                    acc = fmaf(w[j].x, t_in >= 3 ? h[k][j] : 0.f, acc);
                    acc = fmaf(w[j].y, t_in >= 2 ? h[k + 1][j] : 0.f, acc);
                    acc = fmaf(w[j].z, t_in >= 1 ? h[k + 2][j] : 0.f, acc);
                    acc = fmaf(w[j].w, h[k + 3][j], acc);
                    o[j] = silu_fast(acc);
                }
                *reinterpret_cast<uint4 *>(dst + (size_t)r * dst_ld) = pack8(o);
            }
        }
    }
}

}  // namespace

#define STR_DTYPE_OK(dt) ((dt) == STR_F32 || (dt) == STR_BF16)

extern "C" int str_rmsnorm(str_ctx *ctx, int dtype, int rows, int D, float eps, const void *in, void *out,
                           void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !in || !out || rows < 0 || D <= 0 || !STR_DTYPE_OK(dtype)) return STR_ERR_INVALID_ARG;
    if (rows == 0) return STR_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == STR_BF16 && D % 8 == 0 && D <= 32 * 8 * 16 && (((uintptr_t)in | (uintptr_t)out) & 15) == 0)
        rmsnorm_bf16_vec_kernel<16><<<ceil_div(rows, 8), 256, 0, st>>>(rows, D, eps, (const __nv_bfloat16 *)in,
                                                                         (__nv_bfloat16 *)out);
    else if (dtype == STR_BF16)
        rmsnorm_kernel<__nv_bfloat16><<<rows, 256, 0, st>>>(D, eps, (const __nv_bfloat16 *)in, (__nv_bfloat16 *)out);
    else
        rmsnorm_kernel<float><<<rows, 256, 0, st>>>(D, eps, (const float *)in, (float *)out);
    return str_launch_ok(ctx);
}

// Squared ReLU, element-wise (the FFN block's activation); in place when out == in.
template <typename T>
__global__ void __launch_bounds__(256) relu2_kernel(size_t n, const T *__restrict__ in, T *__restrict__ out) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float v = fmaxf(ldf(in + i), 0.f);
        stf(out + i, v * v);
    }
}
__global__ void __launch_bounds__(256) relu2_bf16_vec_kernel(size_t n8, const uint4 *__restrict__ in, uint4 *__restrict__ out) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = in[i];
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float lo = fmaxf(__uint_as_float(w[j] << 16), 0.f), hi = fmaxf(__uint_as_float(w[j] & 0xFFFF0000u), 0.f);
            const __nv_bfloat162 pk = __floats2bfloat162_rn(lo * lo, hi * hi);
            w[j] = *reinterpret_cast<const uint32_t *>(&pk);
        }
        out[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

extern "C" int str_relu_squared(str_ctx *ctx, int dtype, size_t n, const void *in, void *out, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !in || !out || !STR_DTYPE_OK(dtype)) return STR_ERR_INVALID_ARG;
    if (n == 0) return STR_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int cap = ctx->sm_count * 16;
    if (dtype == STR_BF16 && n % 8 == 0 && (((uintptr_t)in | (uintptr_t)out) & 15) == 0) {
        const size_t n8 = n / 8, blocks = (n8 + 255) / 256;
        relu2_bf16_vec_kernel<<<(unsigned)(blocks < (size_t)cap ? blocks : cap), 256, 0, st>>>(n8, (const uint4 *)in, (uint4 *)out);
    } else {
        const size_t blocks = (n + 255) / 256;
        const unsigned g = (unsigned)(blocks < (size_t)cap ? blocks : cap);
        if (dtype == STR_BF16) relu2_kernel<__nv_bfloat16><<<g, 256, 0, st>>>(n, (const __nv_bfloat16 *)in, (__nv_bfloat16 *)out);
        else relu2_kernel<float><<<g, 256, 0, st>>>(n, (const float *)in, (float *)out);
    }
    return str_launch_ok(ctx);
}

// RoPE + split, bf16, 16 bytes per access: one CTA per token row.  The rotation angles depend on the row's
// position and the pair index only, so their sines and cosines (fp64 angle, reduced to [0, 2 pi), as in the
// scalar kernel) are formed once per row in shared memory and shared by all heads; each thread then rotates 8
// pairs (elements i..i+7 of the first half with the matching ones of the second half) or copies 8 v columns.
__global__ void __launch_bounds__(256)
rope_split_bf16_vec_kernel(int Hq, int Hkv, int d, double log2_theta, const int32_t *__restrict__ positions,
                           const __nv_bfloat16 *__restrict__ qkv, __nv_bfloat16 *__restrict__ q_out,
                           __nv_bfloat16 *__restrict__ k_out, __nv_bfloat16 *__restrict__ v_out) {
    extern __shared__ float cs_sn[];                    // [half] cos | [half] sin
    const int half = d / 2, h8 = half / 8;
    const size_t row = blockIdx.x;
    const int ld = (Hq + 2 * Hkv) * d;
    const __nv_bfloat16 *base = qkv + row * ld;
    const double pos = (double)positions[row];
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double inv_freq = exp2(-2.0 * (double)i / (double)d * log2_theta);
        double ang = pos * inv_freq;
        ang -= 6.283185307179586476925 * floor(ang * 0.15915494309189533576888);
        float sn, cs;
        sincosf((float)ang, &sn, &cs);
        cs_sn[i] = cs;
        cs_sn[half + i] = sn;
    }
    __syncthreads();
    const int n_rot = (Hq + Hkv) * h8, n_v = Hkv * d / 8;
    for (int e = threadIdx.x; e < n_rot + n_v; e += blockDim.x) {
        if (e < n_rot) {
            const int head = e / h8, i0 = (e - head * h8) * 8;
            const uint4 va = __ldg(reinterpret_cast<const uint4 *>(base + head * d + i0));
            const uint4 vb = __ldg(reinterpret_cast<const uint4 *>(base + head * d + half + i0));
            float a[8], b[8];
            unpack8(va, a);
            unpack8(vb, b);
            uint32_t oa[4], ob[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float c0 = cs_sn[i0 + 2 * j], s0 = cs_sn[half + i0 + 2 * j];
                const float c1 = cs_sn[i0 + 2 * j + 1], s1 = cs_sn[half + i0 + 2 * j + 1];
                oa[j] = pack2(a[2 * j] * c0 - b[2 * j] * s0, a[2 * j + 1] * c1 - b[2 * j + 1] * s1);
                ob[j] = pack2(b[2 * j] * c0 + a[2 * j] * s0, b[2 * j + 1] * c1 + a[2 * j + 1] * s1);
            }
            __nv_bfloat16 *dst = head < Hq ? q_out + (row * Hq + head) * d : k_out + (row * Hkv + (head - Hq)) * d;
            *reinterpret_cast<uint4 *>(dst + i0) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
            *reinterpret_cast<uint4 *>(dst + half + i0) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
        } else {
            const int c = (e - n_rot) * 8;
            *reinterpret_cast<uint4 *>(v_out + row * (size_t)(Hkv * d) + c) =
                __ldg(reinterpret_cast<const uint4 *>(base + (Hq + Hkv) * d + c));
        }
    }
}

static int launch_gated_rmsnorm(str_ctx *ctx, int dtype, int rows, int d_inner, int ld_z, float eps, const void *y,
                                const void *z, void *out, RowGather rg, cudaStream_t st) {
    if (dtype == STR_BF16 && d_inner % 8 == 0 && ld_z % 8 == 0 && d_inner <= 256 * 8 * 4 &&
        (((uintptr_t)y | (uintptr_t)z | (uintptr_t)out) & 15) == 0)
        gated_rmsnorm_bf16_vec_kernel<4><<<rows, 256, 0, st>>>(d_inner, ld_z, eps, (const __nv_bfloat16 *)y,
                                                                (const __nv_bfloat16 *)z, (__nv_bfloat16 *)out, rg);
    else if (dtype == STR_BF16)
        gated_rmsnorm_kernel<__nv_bfloat16><<<rows, 256, 0, st>>>(d_inner, ld_z, eps, (const __nv_bfloat16 *)y,
                                                                 (const __nv_bfloat16 *)z, (__nv_bfloat16 *)out, rg);
    else
        gated_rmsnorm_kernel<float><<<rows, 256, 0, st>>>(d_inner, ld_z, eps, (const float *)y, (const float *)z,
                                                         (float *)out, rg);
    return str_launch_ok(ctx);
}

extern "C" int str_gated_rmsnorm(str_ctx *ctx, int dtype, int rows, int d_inner, int ld_z, float eps,
                                 const void *y, const void *z, void *out, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !y || !z || !out || rows < 0 || d_inner <= 0 || ld_z < d_inner || !STR_DTYPE_OK(dtype))
        return STR_ERR_INVALID_ARG;
    if (rows == 0) return STR_OK;
    return launch_gated_rmsnorm(ctx, dtype, rows, d_inner, ld_z, eps, y, z, out, RowGather{nullptr, 0, 0, 0, 0, false},
                                (cudaStream_t)stream);
}

// Internal (stack driver): the same operation on gathered rows.  Output row (b, j) takes y and z from input row
// kept[b][j] for j < k and from text row n_vis + (j - k) after that, so the rows a reducing layer is about to
// drop are never normalised or projected.
int str_gated_rmsnorm_gather(str_ctx *ctx, int dtype, int Bz, int T_in, int n_vis, int n_text, int k, int d_inner, int ld_z,
                             float eps, const void *y, const void *z, bool z_compacted, const int32_t *kept, void *out,
                             void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !y || !z || !out || !kept || Bz <= 0 || k < 0 || k > n_vis || T_in != n_vis + n_text || d_inner <= 0 ||
        ld_z < d_inner || !STR_DTYPE_OK(dtype))
        return STR_ERR_INVALID_ARG;
    const int rows = Bz * (k + n_text);
    if (rows == 0) return STR_OK;
    return launch_gated_rmsnorm(ctx, dtype, rows, d_inner, ld_z, eps, y, z, out, RowGather{kept, T_in, n_vis, k, k + n_text, z_compacted},
                                (cudaStream_t)stream);
}

// has_z: rows are [z | x B C | dt_raw]; otherwise [x B C | dt_raw] (the gate columns are projected separately).
int str_mamba_conv_split_rows(str_ctx *ctx, int dtype, int Bz, int T, int H, int p, int n, int G, int W, bool has_z,
                              const void *zxbcdt, const float *conv_w, const float *conv_b, const float *dt_bias,
                              void *x_out, void *B_out, void *C_out, float *dt_out, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !zxbcdt || !conv_w || !conv_b || !dt_bias || !x_out || !B_out || !C_out || !dt_out || Bz <= 0 ||
        T <= 0 || H <= 0 || p <= 0 || n <= 0 || G <= 0 || W <= 0 || !STR_DTYPE_OK(dtype))
        return STR_ERR_INVALID_ARG;
    if ((long long)Bz * T > 2147483647LL) return STR_ERR_UNSUPPORTED_SHAPE;
    const int cols = H * p + 2 * G * n + H;
    dim3 grid(Bz * T, ceil_div(cols, 256));
    cudaStream_t st = (cudaStream_t)stream;
    const int d_inner_ = H * p, gn_ = G * n;
    const int zoff = has_z ? d_inner_ : 0;
    if (dtype == STR_BF16 && W == 4 && d_inner_ % 8 == 0 && gn_ % 8 == 0 && H % 8 == 0 &&
        (((uintptr_t)zxbcdt | (uintptr_t)x_out | (uintptr_t)B_out | (uintptr_t)C_out | (uintptr_t)conv_w) & 15) == 0) {
        const int tiles = ceil_div(T, CONV_TT);
        dim3 vgrid(Bz * tiles, ceil_div((d_inner_ + 2 * gn_) / CONV_CPT, 256) + 1);
        mamba_conv_split_bf16_vec_kernel<<<vgrid, 256, 0, st>>>(
            T, H, p, n, G, zoff, (const __nv_bfloat16 *)zxbcdt, conv_w, conv_b, dt_bias, (__nv_bfloat16 *)x_out,
            (__nv_bfloat16 *)B_out, (__nv_bfloat16 *)C_out, dt_out);
        return str_launch_ok(ctx);
    }
    if (dtype == STR_BF16)
        mamba_conv_split_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
            T, H, p, n, G, W, zoff, (const __nv_bfloat16 *)zxbcdt, conv_w, conv_b, dt_bias, (__nv_bfloat16 *)x_out,
            (__nv_bfloat16 *)B_out, (__nv_bfloat16 *)C_out, dt_out);
    else
        mamba_conv_split_kernel<float><<<grid, 256, 0, st>>>(T, H, p, n, G, W, zoff, (const float *)zxbcdt, conv_w, conv_b,
                                                            dt_bias, (float *)x_out, (float *)B_out, (float *)C_out,
                                                            dt_out);
    return str_launch_ok(ctx);
}

int str_mamba_conv_edge_rows(str_ctx *ctx, int Bz, int T, int ld, const StrConvEpilogue &cv, const void *zxbcdt, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    const long long rows = (long long)Bz * T;
    if (rows <= 0 || rows > 2147483647LL) return STR_ERR_INVALID_ARG;
    dim3 grid(ceil_div(ceil_div((int)rows, 32), EDGE_GROUPS), ceil_div((cv.d_inner + 2 * cv.gn) / 8, 256));
    mamba_conv_edge_rows_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((int)rows, T, ld, cv.zoff, cv.d_inner, cv.gn,
                                                                       (const __nv_bfloat16 *)zxbcdt, cv.conv_w, cv.conv_b,
                                                                       cv.x_out, cv.B_out, cv.C_out);
    return str_launch_ok(ctx);
}

extern "C" int str_mamba_conv_split(str_ctx *ctx, int dtype, int Bz, int T, int H, int p, int n, int G, int W,
                                    const void *zxbcdt, const float *conv_w, const float *conv_b,
                                    const float *dt_bias, void *x_out, void *B_out, void *C_out, float *dt_out,
                                    void *stream) {
    return str_mamba_conv_split_rows(ctx, dtype, Bz, T, H, p, n, G, W, true, zxbcdt, conv_w, conv_b, dt_bias, x_out, B_out,
                                     C_out, dt_out, stream);
}

extern "C" int str_rope_split(str_ctx *ctx, int dtype, int Bz, int T, int Hq, int Hkv, int d, float theta,
                              const int32_t *positions, const void *qkv, void *q_out, void *k_out, void *v_out,
                              void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_ELEMENTWISE, stream);
    if (!ctx || !positions || !qkv || !q_out || !k_out || !v_out || Bz <= 0 || T <= 0 || Hq <= 0 || Hkv <= 0 ||
        d <= 0 || (d & 1) || theta <= 0.f || !STR_DTYPE_OK(dtype))
        return STR_ERR_INVALID_ARG;
    if ((long long)Bz * T > 2147483647LL) return STR_ERR_UNSUPPORTED_SHAPE;
    const int work = (Hq + Hkv) * (d / 2) + Hkv * d;
    dim3 grid(Bz * T, ceil_div(work, 256));
    cudaStream_t st = (cudaStream_t)stream;
    const double l2t = log2((double)theta);
    if (dtype == STR_BF16 && d % 16 == 0 && d <= 8192 &&
        (((uintptr_t)qkv | (uintptr_t)q_out | (uintptr_t)k_out | (uintptr_t)v_out) & 15) == 0)
        rope_split_bf16_vec_kernel<<<Bz * T, 256, (size_t)d * sizeof(float), st>>>(
            Hq, Hkv, d, l2t, positions, (const __nv_bfloat16 *)qkv, (__nv_bfloat16 *)q_out, (__nv_bfloat16 *)k_out,
            (__nv_bfloat16 *)v_out);
    else if (dtype == STR_BF16)
        rope_split_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(Hq, Hkv, d, l2t, positions, (const __nv_bfloat16 *)qkv,
                                                              (__nv_bfloat16 *)q_out, (__nv_bfloat16 *)k_out,
                                                              (__nv_bfloat16 *)v_out);
    else
        rope_split_kernel<float><<<grid, 256, 0, st>>>(Hq, Hkv, d, l2t, positions, (const float *)qkv, (float *)q_out,
                                                      (float *)k_out, (float *)v_out);
    return str_launch_ok(ctx);
}
