// Mamba-2 SSD chunked scan on tcgen05 tensor cores (bf16 in, fp32 accumulate), head dim p = 64,
// state dim n = 128.  One CTA per (sequence, head) walks the sequence in chunks of 128 tokens and
// carries the running state in registers, so chunk states never travel through global memory.
//
// Per chunk, with l_t the in-chunk inclusive cumulative log-decay (l_t = sum_{u<=t} dt_u A_h <= 0):
//   CB      = C B^T                                  [128 x 128]   tcgen05, K-major operands
//   W[t,j]  = CB[t,j] exp(l_t - l_j) dt_j 1[j<=t]    fp32 on CUDA cores -> bf16 -> shared memory
//   Y_intra = W X                                    [128 x 64]    tcgen05, X as MN-major operand
//   Y_inter = C S_prev^T                             [128 x 64]    tcgen05, bf16 copy of the state
//   y_t     = Y_intra[t] + exp(l_t) Y_inter[t]                     fp32 epilogue -> bf16 -> global
//   dS^T    = B^T Xs,  Xs_j = exp(l_end - l_j) dt_j x_j  [128 x 64] tcgen05, both operands MN-major
//   S^T    <- exp(l_end) S^T + dS^T                                fp32 registers (the master state)
// Every decay factor is formed from a difference of cumulative sums that is <= 0.  Off the
// diagonal 32x32 blocks exp(l_t - l_j) is split into three factors, each <= 1 (row part, block-pair
// scalar, column part), which turns 128x128 exponentials per chunk into O(128) plus the diagonal blocks.
//
// Warp roles: 0-7 compute (256 threads; warp w owns TMEM lane quadrant w%4 and column half w/4),
// 8 = TMA producer (x, B, C tiles, 128-byte swizzle, 2 stages), 9 = MMA issuer (one thread).
// All mbarrier waits are bounded; a give-up records STR_ERR_TIMEOUT and tears the CTA down.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int Q = 128, P = 64, NS = 128;
constexpr int TILE_16K = 16384;
constexpr int OFF_X = 0, OFF_B = TILE_16K, OFF_C = 3 * TILE_16K, STAGE_BYTES = 5 * TILE_16K;   // X | B0 B1 | C0 C1
constexpr int OFF_W = 2 * STAGE_BYTES, OFF_XT = OFF_W + 2 * TILE_16K, OFF_SB = OFF_XT + TILE_16K;
constexpr int OFF_MISC = OFF_SB + TILE_16K;
constexpr int MISC_BYTES = 4 * 512 + 32 + 64 + 14 * 8 + 16;
constexpr size_t SMEM_BYTES = (size_t)OFF_MISC + MISC_BYTES;
constexpr int COMPUTE_THREADS = 256, NUM_THREADS = 320;
// TMEM columns
constexpr uint32_t TM_CB = 0, TM_YI = 256, TM_YO = 320, TM_DS = 384;

enum { B_FULL0 = 0, B_FULL1, B_EMPTY0, B_EMPTY1, B_CBR0, B_CBR1, B_CBF0, B_CBF1, B_XT, B_DS, B_W, B_S, B_Y, B_YF, B_COUNT };

__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// Barrier over the 256 compute threads that also ANDs a predicate, so that every compute warp takes
// the same decision to leave the chunk loop (a warp that left alone would strand the others).
__device__ __forceinline__ bool compute_sync_and(bool v) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)v) : "memory");
    return r != 0;
}

__device__ __forceinline__ void warp_arrive(uint64_t *bar, int lane) {
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(bar);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
ssd_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
              const __grid_constant__ CUtensorMap tmap_c, int Tlen, int H, int G, const float *__restrict__ dt,
              const float *__restrict__ A, __nv_bfloat16 *__restrict__ y, float *__restrict__ final_state, int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *misc = smem + OFF_MISC;
    float *ls = (float *)misc;            // [128] cumulative log-decay
    float *dts = ls + 128;                // [128] dt
    float *colf = dts + 128;              // [128] exp(l_blockend - l_j) * dt_j
    float *xw = colf + 128;               // [128] exp(l_end - l_j) * dt_j
    float *wsum = xw + 128;               // [4] per-block sums of dt*A, then [4] block-start values
    float *blk = wsum + 8;                // [4][4] exp(l_blockstart(bt) - l_blockend(bj))
    uint64_t *bars = (uint64_t *)(blk + 16);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.x, b = blockIdx.y, g = h / (H / G);
    const int nchunks = (Tlen + Q - 1) / Q;

    if ((tc::smem_u32(smem) & 1023u) != 0) {          // swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    if (threadIdx.x == 0) {
        tc::mbar_init(bars + B_FULL0, 1); tc::mbar_init(bars + B_FULL1, 1);
        tc::mbar_init(bars + B_EMPTY0, 1); tc::mbar_init(bars + B_EMPTY1, 1);
        tc::mbar_init(bars + B_CBR0, 1); tc::mbar_init(bars + B_CBR1, 1);
        tc::mbar_init(bars + B_CBF0, 8); tc::mbar_init(bars + B_CBF1, 8);
        tc::mbar_init(bars + B_XT, 8); tc::mbar_init(bars + B_DS, 1); tc::mbar_init(bars + B_W, 8);
        tc::mbar_init(bars + B_S, 8); tc::mbar_init(bars + B_Y, 1); tc::mbar_init(bars + B_YF, 8);
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_x); tc::prefetch_tmap(&tmap_b); tc::prefetch_tmap(&tmap_c);
    }
    if (warp == 9) { tc::tmem_alloc(tmem_slot, 512); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            int c = 0;
            for (; c < nchunks; ++c) {
                const int s = c & 1;
                if (!tc::mbar_wait(bars + B_EMPTY0 + s, ((c >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
                uint64_t *fb = bars + B_FULL0 + s;
                tc::mbar_arrive_expect_tx(fb, STAGE_BYTES);
                uint8_t *st = smem + (size_t)s * STAGE_BYTES;
                const int t0 = c * Q;
                tc::tma_load_3d(st + OFF_X, &tmap_x, fb, h * P, t0, b);
                tc::tma_load_3d(st + OFF_B, &tmap_b, fb, g * NS, t0, b);
                tc::tma_load_3d(st + OFF_B + TILE_16K, &tmap_b, fb, g * NS + 64, t0, b);
                tc::tma_load_3d(st + OFF_C, &tmap_c, fb, g * NS, t0, b);
                tc::tma_load_3d(st + OFF_C + TILE_16K, &tmap_c, fb, g * NS + 64, t0, b);
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                for (int back = 1; back <= 2 && back <= c; ++back) {      // let issued copies land
                    const int j = c - back;
                    tc::mbar_wait(bars + B_FULL0 + (j & 1), (j >> 1) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t id_cb = tc::make_idesc_bf16(128, 128, 0, 0);   // C (K-major) x B (K-major)
            const uint32_t id_kn = tc::make_idesc_bf16(128, 64, 0, 1);    // K-major A x MN-major B
            const uint32_t id_nn = tc::make_idesc_bf16(128, 64, 1, 1);    // MN-major A x MN-major B
            const uint32_t sbase = tc::smem_u32(smem);
            bool ok = true;
            auto issue_cb = [&](int c) {
                const uint32_t st = sbase + (uint32_t)(c & 1) * STAGE_BYTES;
                const uint32_t d = tmem + TM_CB + (uint32_t)(c & 1) * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc::mma_ss(d, tc::desc_kmajor_sw128(st + OFF_C + (ks >> 2) * TILE_16K, (ks & 3) * 16),
                               tc::desc_kmajor_sw128(st + OFF_B + (ks >> 2) * TILE_16K, (ks & 3) * 16), id_cb, ks != 0);
                tc::mma_commit(bars + B_CBR0 + (c & 1));
            };
            if (nchunks > 0) {
                ok = tc::mbar_wait(bars + B_FULL0, 0, abort_flag);
                if (ok) { tc::tc_fence_after(); issue_cb(0); }
            }
            for (int c = 0; c < nchunks && ok; ++c) {
                const uint32_t st = sbase + (uint32_t)(c & 1) * STAGE_BYTES;
                if (c > 0) {
                    // state of chunk c-1 is in shared memory; Y accumulators have been read out
                    if (!tc::mbar_wait(bars + B_S, (c - 1) & 1, abort_flag)) { ok = false; break; }
                    if (!tc::mbar_wait(bars + B_YF, (c - 1) & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)      // Y_inter = C S_prev^T
                        tc::mma_ss(tmem + TM_YO, tc::desc_kmajor_sw128(st + OFF_C + (ks >> 2) * TILE_16K, (ks & 3) * 16),
                                   tc::make_smem_desc(sbase + OFF_SB + ks * 2048, TILE_16K, 1024, tc::SWZ_128B), id_kn,
                                   ks != 0);
                }
                if (!tc::mbar_wait(bars + B_XT, c & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)          // dS^T = B^T Xs
                    tc::mma_ss(tmem + TM_DS, tc::make_smem_desc(st + OFF_B + ks * 2048, TILE_16K, 1024, tc::SWZ_128B),
                               tc::make_smem_desc(sbase + OFF_XT + ks * 2048, TILE_16K, 1024, tc::SWZ_128B), id_nn,
                               ks != 0);
                tc::mma_commit(bars + B_DS);
                if (c + 1 < nchunks) {
                    const int nb = (c + 1) & 1;
                    if (!tc::mbar_wait(bars + B_FULL0 + nb, ((c + 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    if (c >= 1 && !tc::mbar_wait(bars + B_CBF0 + nb, ((c - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    issue_cb(c + 1);
                }
                if (!tc::mbar_wait(bars + B_W, c & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)          // Y_intra = W X
                    tc::mma_ss(tmem + TM_YI, tc::desc_kmajor_sw128(sbase + OFF_W + (ks >> 2) * TILE_16K, (ks & 3) * 16),
                               tc::make_smem_desc(st + OFF_X + ks * 2048, TILE_16K, 1024, tc::SWZ_128B), id_kn, ks != 0);
                tc::mma_commit(bars + B_Y);
                tc::mma_commit(bars + B_EMPTY0 + (c & 1));
            }
            if (!ok) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ compute warps
        const int tid = threadIdx.x;                  // 0..255
        const int quad = warp & 3, hf = warp >> 2;
        const int row = quad * 32 + lane;             // token (W, Y) or state index n (state)
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const float Ah = A[h];
        const float *dtb = dt + (size_t)b * Tlen * H + h;
        __nv_bfloat16 *yb = y + ((size_t)b * Tlen * H + h) * P;
        float S[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) S[i] = 0.f;
        bool ok = true;
        for (int c = 0; c < nchunks; ++c) {
            const int s = c & 1, t0 = c * Q;
            uint8_t *st = smem + (size_t)s * STAGE_BYTES;
            // ---- 1. cumulative log-decay and factors
            float a_incl = 0.f, d_me = 0.f;
            if (tid < 128) {
                d_me = (t0 + tid < Tlen) ? dtb[(size_t)(t0 + tid) * H] : 0.f;
                a_incl = d_me * Ah;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float v = __shfl_up_sync(0xffffffffu, a_incl, o);
                    if (lane >= o) a_incl += v;
                }
                if (lane == 31) wsum[warp] = a_incl;
            }
            ok = compute_sync_and(ok);       // uniform: a failed wait anywhere ends the loop for all warps
            if (!ok) break;
            if (tid < 128) {
                float l_start = 0.f;
                for (int w = 0; w < warp; ++w) l_start += wsum[w];
                const float l_end_blk = l_start + wsum[warp];
                const float l_end = wsum[0] + wsum[1] + wsum[2] + wsum[3];
                const float l = l_start + a_incl;
                ls[tid] = l;
                dts[tid] = d_me;
                colf[tid] = __expf(l_end_blk - l) * d_me;
                xw[tid] = __expf(l_end - l) * d_me;
                if (lane == 0) wsum[4 + warp] = l_start;
                if (lane < 4 && lane < warp) {            // blk[bt = warp][bj = lane], bj < bt
                    float l_end_bj = 0.f;
                    for (int w = 0; w <= lane; ++w) l_end_bj += wsum[w];
                    blk[warp * 4 + lane] = __expf(l_start - l_end_bj);
                }
            }
            ok &= tc::mbar_wait(bars + B_FULL0 + s, (c >> 1) & 1, abort_flag);
            compute_sync();
            // ---- 2. Xs = exp(l_end - l_j) dt_j x_j  (same swizzled layout as the X tile)
            {
                const uint4 *src = (const uint4 *)(st + OFF_X);
                uint4 *dst = (uint4 *)(smem + OFF_XT);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int u = tid + 256 * i;
                    const float sc = xw[u >> 3];
                    uint4 v = src[u];
                    uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        wv[j] = tc::pack_bf16x2(__uint_as_float(wv[j] << 16) * sc, __uint_as_float(wv[j] & 0xFFFF0000u) * sc);
                    dst[u] = make_uint4(wv[0], wv[1], wv[2], wv[3]);
                }
            }
            tc::fence_proxy_async();
            warp_arrive(bars + B_XT, lane);
            // ---- 3. W = CB o decay (bf16, K-major swizzled tile; this warp: rows of block `quad`, 64 columns)
            ok &= tc::mbar_wait(bars + B_CBR0 + s, (c >> 1) & 1, abort_flag);
            tc::tc_fence_after();
            {
                const float l_t = ls[row], rf = __expf(l_t - wsum[4 + quad]);
                uint8_t *wrow = smem + OFF_W + hf * TILE_16K + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
                for (int cg = 0; cg < 2; ++cg) {
                    const int bj = 2 * hf + cg;
                    uint32_t packed[16];
                    if (bj > quad) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) packed[i] = 0u;
                    } else {
                        uint32_t v[32];
                        tc::tmem_ld32(tmem + lane_base + TM_CB + (uint32_t)s * 128 + (uint32_t)(bj * 32), v);
                        tc::tmem_ld_wait();
                        if (bj == quad) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int j0 = bj * 32 + 2 * i, j1 = j0 + 1;
                                const float f0 = (j0 <= row) ? __expf(l_t - ls[j0]) * dts[j0] : 0.f;
                                const float f1 = (j1 <= row) ? __expf(l_t - ls[j1]) * dts[j1] : 0.f;
                                packed[i] = tc::pack_bf16x2(__uint_as_float(v[2 * i]) * f0, __uint_as_float(v[2 * i + 1]) * f1);
                            }
                        } else {
                            const float f = rf * blk[quad * 4 + bj];
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int j0 = bj * 32 + 2 * i;
                                packed[i] = tc::pack_bf16x2(__uint_as_float(v[2 * i]) * (f * colf[j0]),
                                                            __uint_as_float(v[2 * i + 1]) * (f * colf[j0 + 1]));
                            }
                        }
                    }
#pragma unroll
                    for (int ci = 0; ci < 4; ++ci) {
                        const int chunk = cg * 4 + ci;
                        *(uint4 *)(wrow + ((chunk ^ (row & 7)) << 4)) =
                            make_uint4(packed[4 * ci], packed[4 * ci + 1], packed[4 * ci + 2], packed[4 * ci + 3]);
                    }
                }
            }
            tc::tc_fence_before();
            tc::fence_proxy_async();
            warp_arrive(bars + B_W, lane);
            warp_arrive(bars + B_CBF0 + s, lane);
            // ---- 4. state: S^T <- exp(l_end) S^T + dS^T ; bf16 copy for the next chunk's Y_inter
            ok &= tc::mbar_wait(bars + B_DS, c & 1, abort_flag);
            tc::tc_fence_after();
            {
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + TM_DS + (uint32_t)(hf * 32), v);
                tc::tmem_ld_wait();
                const float eend = __expf(ls[127]);
#pragma unroll
                for (int i = 0; i < 32; ++i) S[i] = fmaf(eend, S[i], __uint_as_float(v[i]));
                uint8_t *srow = smem + OFF_SB + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
                for (int ci = 0; ci < 4; ++ci) {
                    const int chunk = hf * 4 + ci;
                    *(uint4 *)(srow + ((chunk ^ (row & 7)) << 4)) =
                        make_uint4(tc::pack_bf16x2(S[8 * ci], S[8 * ci + 1]), tc::pack_bf16x2(S[8 * ci + 2], S[8 * ci + 3]),
                                   tc::pack_bf16x2(S[8 * ci + 4], S[8 * ci + 5]), tc::pack_bf16x2(S[8 * ci + 6], S[8 * ci + 7]));
                }
            }
            tc::tc_fence_before();
            tc::fence_proxy_async();
            warp_arrive(bars + B_S, lane);
            // ---- 5. epilogue: y_t = Y_intra + exp(l_t) Y_inter
            ok &= tc::mbar_wait(bars + B_Y, c & 1, abort_flag);
            tc::tc_fence_after();
            {
                uint32_t yi[32];
                tc::tmem_ld32(tmem + lane_base + TM_YI + (uint32_t)(hf * 32), yi);
                float out[32];
                if (c > 0) {
                    uint32_t yo[32];
                    tc::tmem_ld32(tmem + lane_base + TM_YO + (uint32_t)(hf * 32), yo);
                    tc::tmem_ld_wait();
                    const float er = __expf(ls[row]);
#pragma unroll
                    for (int i = 0; i < 32; ++i) out[i] = fmaf(er, __uint_as_float(yo[i]), __uint_as_float(yi[i]));
                } else {
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) out[i] = __uint_as_float(yi[i]);
                }
                if (t0 + row < Tlen) {
                    uint4 *dst = (uint4 *)(yb + (size_t)(t0 + row) * H * P + hf * 32);
#pragma unroll
                    for (int ci = 0; ci < 4; ++ci)
                        dst[ci] = make_uint4(tc::pack_bf16x2(out[8 * ci], out[8 * ci + 1]), tc::pack_bf16x2(out[8 * ci + 2], out[8 * ci + 3]),
                                             tc::pack_bf16x2(out[8 * ci + 4], out[8 * ci + 5]), tc::pack_bf16x2(out[8 * ci + 6], out[8 * ci + 7]));
                }
            }
            tc::tc_fence_before();
            warp_arrive(bars + B_YF, lane);
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        if (ok && final_state) {
            float *fs = final_state + ((size_t)b * H + h) * P * NS;
#pragma unroll
            for (int i = 0; i < 32; ++i) fs[(size_t)(hf * 32 + i) * NS + row] = S[i];
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 9) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 512); }
}

int make_tmap_3d(str_ctx *ctx, CUtensorMap *map, const void *base, uint64_t inner, uint64_t T, uint64_t Bz) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    if (!ctx->encode_tiled) return STR_ERR_CUDA;
    cuuint64_t dims[3] = {inner, T, Bz};
    cuuint64_t strides[2] = {inner * 2, inner * T * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)Q, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((encode_fn)ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims,
                                                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? STR_OK : STR_ERR_CUDA;
}

}  // namespace

bool str_ssd_tc_supported(const str_ssd_shape *s, const void *x, const void *B, const void *C, const void *y,
                          const float *D, const float *init_state) {
    if (s->dtype != STR_BF16 || s->p != P || s->n != NS || D || init_state || s->T < 1) return false;
    return (((uintptr_t)x | (uintptr_t)B | (uintptr_t)C | (uintptr_t)y) & 15) == 0;
}

int str_ssd_tc(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt, const float *A, const void *B,
               const void *C, void *y, float *final_state, cudaStream_t st) {
    if (SMEM_BYTES > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tx, tb, tcm;
    int rc = make_tmap_3d(ctx, &tx, x, (uint64_t)s->H * P, (uint64_t)s->T, (uint64_t)s->Bz);
    if (rc == STR_OK) rc = make_tmap_3d(ctx, &tb, B, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz);
    if (rc == STR_OK) rc = make_tmap_3d(ctx, &tcm, C, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz);
    if (rc != STR_OK) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        STR_CUDA_OK(cudaFuncSetAttribute(ssd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
        attr_set = true;
    }
    dim3 grid(s->H, s->Bz);
    ssd_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tx, tb, tcm, s->T, s->H, s->G, dt, A, (__nv_bfloat16 *)y,
                                                        final_state, ctx->status_dev);
    return str_launch_ok(ctx);
}
