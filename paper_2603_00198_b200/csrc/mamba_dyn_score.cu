// "Full Mamba Dynamic" importance score (Section 3.1, Eq. 1): content alignment times the cumulative decay
// between visual token i and text position t_m = n_vis + m, averaged over text positions and heads,
//   s_i = 1/(M H) sum_{m,h} exp(L_{t_m}^h - L_i^h) dt_{i,h} | b_i^{g(h)} . c_{t_m}^{g(h)} |,   L_t^h = sum_{u<=t} dt_{u,h} A_h.
// The decay is split at the last visual token v = n_vis - 1 so that both factors are <= 1:
//   exp(L_t - L_i) = exp(R_i) exp(F_m),   R_i = sum_{u=i+1..v} a_u <= 0,   F_m = sum_{u=v+1..t_m} a_u <= 0,   a_u = dt_u A_h
// and the score becomes, per group g, a row sum of |P| o D with two small products
//   P = B_vis C_text^T  [n_vis x M]  (the product of Eq. 2)      D = U V^T  [n_vis x M],  U[i,h] = dt_{i,h} exp(R_i^h), V[m,h] = exp(F_m^h)
// over the heads h of the group.  R is a suffix sum taken backwards from v, so it is most accurate where the
// score is largest; far from the text the factor underflows to zero, which is what this score does by design.
//
// This file: the decay-weight pass (chunk sums, super-chunk sums, then suffix walk) and the plain fp32 scoring kernel.  The
// tensor-core scoring kernel is in mamba_dyn_score_tc.cu and reads U, V as bf16 high/low pairs.
#include "common.cuh"
#include "dispatch.cuh"

namespace {

constexpr int CHUNK = 64;          // tokens per block of the decay pass (held in registers by the suffix walk)
constexpr int SUPER = 32;          // chunks per super-chunk: suffix offsets cost nch/SUPER + SUPER loads, not nch

// part[b][chunk][h] = sum of dt[i,h] A_h over the visual tokens of the chunk
__global__ void decay_chunk_sums_kernel(int Tlen, int H, int n_vis, const float *__restrict__ dt, const float *__restrict__ A,
                                        float *__restrict__ part) {
    const int b = blockIdx.y, ch = blockIdx.x, nch = gridDim.x;
    const int i0 = ch * CHUNK, i1 = min(n_vis, i0 + CHUNK);
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        const float *p = dt + ((size_t)b * Tlen + i0) * H + h;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        int i = i0;
        for (; i + 4 <= i1; i += 4, p += 4 * (size_t)H) {
            s0 += __ldg(p); s1 += __ldg(p + H); s2 += __ldg(p + 2 * (size_t)H); s3 += __ldg(p + 3 * (size_t)H);
        }
        for (; i < i1; ++i, p += H) s0 += __ldg(p);
        part[((size_t)b * nch + ch) * H + h] = ((s0 + s1) + (s2 + s3)) * A[h];
    }
}

// sup[b][sc][h] = sum of the chunk sums of super-chunk sc (SUPER consecutive chunks)
__global__ void decay_super_sums_kernel(int H, int nch, const float *__restrict__ part, float *__restrict__ sup) {
    const int b = blockIdx.y, sc = blockIdx.x, nsc = gridDim.x;
    const int c0 = sc * SUPER, c1 = min(nch, c0 + SUPER);
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        float s = 0.f;
        for (int c = c1 - 1; c >= c0; --c) s += part[((size_t)b * nch + c) * H + h];
        sup[((size_t)b * nsc + sc) * H + h] = s;
    }
}

// Output layouts of the decay-weight pass.
//   fp32:  U [Bz, n_vis, H], V [Bz, n_text, H]
//   split: U [Bz, n_vis, G, 64] bf16, V [Bz, n_pad, G, 64] bf16 with, for head j of the group (hpg heads, 3 hpg <= 64),
//          U columns  j: hi(u)   hpg + j: hi(u)   2 hpg + j: lo(u)      V columns  j: hi(v)   hpg + j: lo(v)   2 hpg + j: hi(v)
//          (hi = bf16 rounding, lo = bf16 rounding of the remainder), so that one bf16 product over 3 hpg columns
//          gives hi hi + hi lo + lo hi = u v to about 2^-16; rows n_text..n_pad and the columns up to the next
//          multiple of 16 are zero, columns beyond that are never read.
struct SplitStore {
    __nv_bfloat16 *U, *V;
    int G, hpg;
    __device__ void store(__nv_bfloat16 *row, int j, float val, bool is_v) const {
        const __nv_bfloat16 hi = __float2bfloat16_rn(val);
        const __nv_bfloat16 lo = __float2bfloat16_rn(val - __bfloat162float(hi));
        row[j] = hi;
        row[hpg + j] = is_v ? lo : hi;
        row[2 * hpg + j] = is_v ? hi : lo;
        // columns up to the next multiple of 16 are read by the product's last K step and must be zero
        if (j == 0)
            for (int c = 3 * hpg; c < (3 * hpg + 15) / 16 * 16; ++c) row[c] = __float2bfloat16_rn(0.f);
    }
};

// sum of p[c * stride] for c in [c0, c1), eight loads in flight at a time
__device__ __forceinline__ float suffix_sum(const float *__restrict__ p, int stride, int c0, int c1) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int c = c0;
    for (; c + 8 <= c1; c += 8) {
        float t[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) t[q] = p[(size_t)(c + q) * stride];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] += t[q];
    }
    for (; c < c1; ++c) acc[c & 7] += p[(size_t)c * stride];
    return ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
}

// Blocks 0..nch-1: one chunk of visual tokens each; blocks nch..: one chunk of text rows each.  The chunk's dt
// tile [CHUNK][H] is staged in shared memory with every load in flight at once; then thread h walks its column
// (backwards for the suffix sums R, forwards for the text prefix F).  Dynamic shared memory: CHUNK * H floats.
template <bool SPLIT>
__global__ void __launch_bounds__(256)
decay_weights_kernel(int Tlen, int H, int G, int n_vis, int n_text, int n_pad, int nch, const float *__restrict__ dt,
                     const float *__restrict__ A, const float *__restrict__ part, const float *__restrict__ sup,
                     float *__restrict__ Uf, float *__restrict__ Vf, SplitStore sp) {
    extern __shared__ __align__(16) float tile[];     // [CHUNK][H]
    const int b = blockIdx.y, ch = blockIdx.x;
    const int hpg = H / G;
    const bool text = ch >= nch;
    const int r0 = text ? n_vis + (ch - nch) * CHUNK : ch * CHUNK;         // first row of the chunk
    const int r1 = text ? min(n_vis + n_text, r0 + CHUNK) : min(n_vis, r0 + CHUNK);
    const int nrow = max(r1 - r0, 0);
    {   // stage the tile, eight loads per thread in flight (16-byte loads when the rows allow)
        const float *src = dt + ((size_t)b * Tlen + r0) * H;
        const int n = nrow * H, bd = blockDim.x;
        if ((H & 3) == 0 && (reinterpret_cast<uintptr_t>(dt) & 15) == 0) {
            const float4 *s4 = reinterpret_cast<const float4 *>(src);
            float4 *d4 = reinterpret_cast<float4 *>(tile);
            for (int e0 = threadIdx.x; e0 < n / 4; e0 += 8 * bd) {
                float4 t[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) t[q] = (e0 + q * bd < n / 4) ? __ldg(s4 + e0 + q * bd) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q = 0; q < 8; ++q) if (e0 + q * bd < n / 4) d4[e0 + q * bd] = t[q];
            }
        } else {
            for (int e0 = threadIdx.x; e0 < n; e0 += 8 * bd) {
                float t[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) t[q] = (e0 + q * bd < n) ? __ldg(src + e0 + q * bd) : 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) if (e0 + q * bd < n) tile[e0 + q * bd] = t[q];
            }
        }
    }
    __syncthreads();
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        const float Ah = A[h];
        const int g = h / hpg, j = h - g * hpg;
        if (!text) {
            // R at the chunk's last token = decay of every later visual token
            const int sc = ch / SUPER, nsc = (nch + SUPER - 1) / SUPER;
            float R = suffix_sum(sup + (size_t)b * nsc * H + h, H, sc + 1, nsc) +
                      suffix_sum(part + (size_t)b * nch * H + h, H, ch + 1, min(nch, (sc + 1) * SUPER));
            for (int k = nrow - 1; k >= 0; --k) {
                const int i = r0 + k;
                const float d = tile[k * H + h];
                const float u = d * expf(R);
                if (SPLIT) sp.store(sp.U + (((size_t)b * n_vis + i) * G + g) * 64, j, u, false);
                else Uf[((size_t)b * n_vis + i) * H + h] = u;
                R = fmaf(d, Ah, R);                 // R_{i-1} = R_i + a_i
            }
        } else {
            // F = inclusive prefix of a from the first text row on (a text row's own decay counts); earlier text
            // chunks (at most a few) are summed directly
            float F = suffix_sum(dt + ((size_t)b * Tlen + n_vis) * H + h, H, 0, r0 - n_vis) * Ah;
            const int m0 = r0 - n_vis, rows = SPLIT ? n_pad : n_text;
            for (int k = 0; k < CHUNK && m0 + k < rows; ++k) {
                float v = 0.f;
                if (k < nrow) {
                    F = fmaf(tile[k * H + h], Ah, F);
                    v = expf(F);
                }
                if (SPLIT) sp.store(sp.V + (((size_t)b * n_pad + m0 + k) * G + g) * 64, j, v, true);
                else Vf[((size_t)b * n_text + m0 + k) * H + h] = v;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ plain fp32 scoring
constexpr int TI = 64;        // visual tokens per CTA tile
constexpr int TM = 16;        // text rows per inner block
constexpr int THREADS = 256;  // = TI * 4 row groups; each thread: 1 token x 4 text rows

template <typename T>
__global__ void __launch_bounds__(THREADS)
mamba_dyn_importance_kernel(int Tlen, int H, int n, int G, int n_vis, int n_text, const T *__restrict__ B,
                            const T *__restrict__ C, const float *__restrict__ U, const float *__restrict__ V,
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
    const int i = i0 + ti;
    const float *Ui = U + ((size_t)b * n_vis + min(i, n_vis - 1)) * H;
    const float *Vb = V + (size_t)b * n_text * H;
    float total = 0.f;
    for (int g = 0; g < G; ++g) {
        __syncthreads();
        for (int e = tid; e < TI * n; e += THREADS) {
            const int r = e / n, c = e % n;
            Bs[r * ldk + c] = (i0 + r < n_vis) ? ldf(Bb + ((size_t)(i0 + r) * G + g) * n + c) : 0.f;
        }
        for (int m0 = 0; m0 < n_text; m0 += TM) {
            __syncthreads();
            for (int e = tid; e < TM * n; e += THREADS) {
                const int r = e / n, c = e % n;
                Cs[r * ldk + c] = (m0 + r < n_text) ? ldf(Cb + ((size_t)(n_vis + m0 + r) * G + g) * n + c) : 0.f;
            }
            __syncthreads();
            float d[4] = {0.f, 0.f, 0.f, 0.f};
            const float *bp = Bs + ti * ldk;
            const float *cp = Cs + (rg * 4) * ldk;
            for (int c = 0; c < n; ++c) {
                const float bv = bp[c];
#pragma unroll
                for (int r = 0; r < 4; ++r) d[r] = fmaf(bv, cp[r * ldk + c], d[r]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int m = m0 + rg * 4 + r;
                if (m < n_text) {
                    float w = 0.f;                    // sum over the group's heads of u_{i,h} v_{m,h}
                    for (int hh = 0; hh < hpg; ++hh) w = fmaf(Ui[g * hpg + hh], Vb[(size_t)m * H + g * hpg + hh], w);
                    total = fmaf(fabsf(d[r]), w, total);
                }
            }
        }
    }
    red[rg * TI + ti] = total;
    __syncthreads();
    if (rg == 0 && i < n_vis)
        scores[(size_t)b * n_vis + i] =
            (red[ti] + red[TI + ti] + red[2 * TI + ti] + red[3 * TI + ti]) / ((float)n_text * (float)H);
}

template <typename T>
int launch_dyn(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C,
               const float *U, const float *V, float *scores, cudaStream_t st) {
    const size_t smem = ((size_t)(TI + TM) * (s->n + 1) + 4 * TI) * sizeof(float);
    if (smem > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    if (smem > 48 * 1024)
        STR_CUDA_OK(cudaFuncSetAttribute(mamba_dyn_importance_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ctx->max_smem_optin));
    dim3 grid(ceil_div(n_vis, TI), s->Bz);
    mamba_dyn_importance_kernel<T><<<grid, THREADS, smem, st>>>(s->T, s->H, s->n, s->G, n_vis, n_text, (const T *)B,
                                                                 (const T *)C, U, V, scores);
    return str_launch_ok(ctx);
}

}  // namespace

size_t str_mamba_dyn_part_bytes(const str_ssm_score_shape *s, int n_vis) {
    const int nch = ceil_div(n_vis, CHUNK);
    return align_up((size_t)s->Bz * (nch + ceil_div(nch, SUPER)) * s->H * sizeof(float), 256);
}

// Decay weights into `U`, `V`: fp32 layout when `split` is false, bf16 high/low layout otherwise.
int str_mamba_dyn_weights(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, int n_pad, const float *dt,
                          const float *A, float *part, void *U, void *V, bool split, cudaStream_t st) {
    const int nch = ceil_div(n_vis, CHUNK);
    const int threads = s->H < 32 ? 32 : (s->H > 256 ? 256 : (s->H + 31) / 32 * 32);
    decay_chunk_sums_kernel<<<dim3(nch, s->Bz), threads, 0, st>>>(s->T, s->H, n_vis, dt, A, part);
    int rc = str_launch_ok(ctx);
    if (rc != STR_OK) return rc;
    float *sup = part + (size_t)s->Bz * nch * s->H;
    decay_super_sums_kernel<<<dim3(ceil_div(nch, SUPER), s->Bz), threads, 0, st>>>(s->H, nch, part, sup);
    rc = str_launch_ok(ctx);
    if (rc != STR_OK) return rc;
    SplitStore sp{(__nv_bfloat16 *)U, (__nv_bfloat16 *)V, s->G, s->H / s->G};
    const size_t tile_bytes = (size_t)CHUNK * s->H * sizeof(float);
    if (tile_bytes > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    const dim3 grid(nch + ceil_div(split ? n_pad : n_text, CHUNK), s->Bz);
    if (split) {
        if (tile_bytes > 48 * 1024)
            STR_CUDA_OK(cudaFuncSetAttribute(decay_weights_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
        decay_weights_kernel<true><<<grid, threads, tile_bytes, st>>>(s->T, s->H, s->G, n_vis, n_text, n_pad, nch, dt, A, part, sup,
                                                                     nullptr, nullptr, sp);
    } else {
        if (tile_bytes > 48 * 1024)
            STR_CUDA_OK(cudaFuncSetAttribute(decay_weights_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
        decay_weights_kernel<false><<<grid, threads, tile_bytes, st>>>(s->T, s->H, s->G, n_vis, n_text, n_pad, nch, dt, A, part, sup,
                                                                      (float *)U, (float *)V, sp);
    }
    return str_launch_ok(ctx);
}

int str_mamba_dyn_importance_simt(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B,
                                  const void *C, const float *U, const float *V, float *scores, cudaStream_t st) {
    return s->dtype == STR_BF16 ? launch_dyn<__nv_bfloat16>(ctx, s, n_vis, n_text, B, C, U, V, scores, st)
                                : launch_dyn<float>(ctx, s, n_vis, n_text, B, C, U, V, scores, st);
}
