// "Full Mamba Dynamic" importance score (Section 3.1, Eq. 1) on tcgen05 tensor cores, bf16 inputs, d_state 128:
//   s_i = 1/(M H) sum_g sum_m | b_i^g . c_m^g |  sum_{h in g} u_{i,h} v_{m,h},
// u_{i,h} = dt_{i,h} exp(R_i^h) and v_{m,h} = exp(F_m^h) the two halves of the cumulative decay between visual
// token i and text row m (see mamba_dyn_score.cu, which writes them as bf16 high/low pairs).  Same persistent
// structure as the Eq. 2 kernel (group outer, tiles inner, running sums in shared memory); per (group, tile)
// two products land in tensor memory,
//   P = B_tile C_text^T   [128 x M], K = 128        D = U_tile V_text^T   [128 x M], K = 3 x heads per group
// and one thread per token row sums |P[i,m]| D[i,m] over m.  D is exact to about 2^-16: its operands carry
// hi(u) hi(v) + hi(u) lo(v) + lo(u) hi(v) along K.
// Warps: 0-3 row sums, 4 TMA producer (B+U ring, two C+V buffers), 5 MMA issuer.  Text rows <= 128 (two
// accumulators of 128 columns per buffer, two buffers).  Every mbarrier wait is bounded.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int TI = 128, NS = 128;
constexpr int B_TILE = 32768;                // 128 tokens x 128 bf16, two 64-column halves
constexpr int U_TILE = 16384;                // 128 tokens x 64 bf16 (3 x heads-per-group columns used)
constexpr int STAGE = B_TILE + U_TILE;
constexpr int MAX_TEXT = 128, MAX_STAGES = 4, MAX_ITEMS = 16;
enum { B_FULL0 = 0, B_EMPTY0 = MAX_STAGES, B_CF0 = 2 * MAX_STAGES, B_CE0 = B_CF0 + 2, B_ACCF0 = B_CE0 + 2, B_ACCE0 = B_ACCF0 + 2,
       B_COUNT = B_ACCE0 + 2 };
constexpr int NUM_THREADS = 192;

__global__ void __launch_bounds__(NUM_THREADS, 1)
mamba_dyn_score_tc_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_c,
                          const __grid_constant__ CUtensorMap tmap_u, const __grid_constant__ CUtensorMap tmap_v, int H, int G,
                          int n_vis, int n_text, int n_pad, int stages, int kd_steps, float *__restrict__ scores, int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int c_only = n_pad * 256;                          // text tile: n_pad rows x 128 bf16 ...
    const int c_bytes = c_only + n_pad * 128;                //            ... followed by its n_pad x 64 decay tile V
    uint8_t *c_smem = smem + stages * STAGE;
    float *totals = (float *)(c_smem + 2 * c_bytes);          // [MAX_ITEMS][128] running sums of this CTA's tiles
    uint64_t *bars = (uint64_t *)(totals + MAX_ITEMS * TI);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int tiles = (n_vis + TI - 1) / TI;
    const int my_tiles = (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;     // tiles of this CTA
    const uint32_t acc_cols = 256u;                            // one buffer: P in columns [0,128), D in [128,256)

    if ((tc::smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    if (tc::cta_should_leave(status)) return;     // an earlier CTA failed: the whole CTA leaves at once
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { tc::mbar_init(bars + B_FULL0 + s, 1); tc::mbar_init(bars + B_EMPTY0 + s, 1); }
        for (int s = 0; s < 2; ++s) {
            tc::mbar_init(bars + B_CF0 + s, 1); tc::mbar_init(bars + B_CE0 + s, 1);
            tc::mbar_init(bars + B_ACCF0 + s, 1); tc::mbar_init(bars + B_ACCE0 + s, 4);
        }
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_b); tc::prefetch_tmap(&tmap_c); tc::prefetch_tmap(&tmap_u); tc::prefetch_tmap(&tmap_v);
    }
    if (warp == 5) { tc::tmem_alloc(tmem_slot, 2 * acc_cols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // All roles walk the same sequence: rounds of up to MAX_ITEMS tiles; inside a round, group g (outer) and
    // tile k (inner).  `it` counts (group, tile) steps and `cg` counts (round, group) steps across the kernel.
    if (warp == 4) {
        if (lane == 0) {
            bool ok = true;
            int it = 0, cg = 0, c_issued = 0;
            for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
                const int kr = min(MAX_ITEMS, my_tiles - r0);
                for (int g = 0; g < G && ok; ++g, ++cg) {
                    const int cs = cg & 1;
                    if (!tc::mbar_wait(bars + B_CE0 + cs, ((cg >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    tc::mbar_arrive_expect_tx(bars + B_CF0 + cs, (uint32_t)c_bytes);
                    tc::tma_load_3d(c_smem + cs * c_bytes, &tmap_c, bars + B_CF0 + cs, g * NS, n_vis, b);
                    tc::tma_load_3d(c_smem + cs * c_bytes + n_pad * 128, &tmap_c, bars + B_CF0 + cs, g * NS + 64, n_vis, b);
                    tc::tma_load_3d(c_smem + cs * c_bytes + c_only, &tmap_v, bars + B_CF0 + cs, g * 64, 0, b);
                    ++c_issued;
                    for (int k = 0; k < kr; ++k, ++it) {
                        const int s = it % stages;
                        if (!tc::mbar_wait(bars + B_EMPTY0 + s, ((it / stages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        const int i0 = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI;
                        uint64_t *fb = bars + B_FULL0 + s;
                        tc::mbar_arrive_expect_tx(fb, STAGE);
                        tc::tma_load_3d(smem + s * STAGE, &tmap_b, fb, g * NS, i0, b);
                        tc::tma_load_3d(smem + s * STAGE + B_TILE / 2, &tmap_b, fb, g * NS + 64, i0, b);
                        tc::tma_load_3d(smem + s * STAGE + B_TILE, &tmap_u, fb, g * 64, i0, b);
                    }
                }
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                // let copies already issued land before the CTA's shared memory goes away
                for (int back = 1; back <= stages && back <= it; ++back) {
                    const int j = it - back;
                    tc::mbar_wait(bars + B_FULL0 + j % stages, (j / stages) & 1, abort_flag + 1);
                }
                for (int back = 1; back <= 2 && back <= c_issued; ++back) {
                    const int j = c_issued - back;
                    tc::mbar_wait(bars + B_CF0 + (j & 1), (j >> 1) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 5) {
        const uint32_t idesc = tc::make_idesc_bf16(TI, n_pad, 0, 0);
        const uint32_t sbase = tc::smem_u32(smem), cbase = tc::smem_u32(c_smem);
        bool ok = true;
        int it = 0, cg = 0;
        for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
            const int kr = min(MAX_ITEMS, my_tiles - r0);
            for (int g = 0; g < G && ok; ++g, ++cg) {
                const int cs = cg & 1;
                ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_CF0 + cs, (cg >> 1) & 1, abort_flag));
                const uint32_t ct = cbase + (uint32_t)(cs * c_bytes);
                for (int k = 0; k < kr && ok; ++k, ++it) {
                    const int s = it & 1, sl = it % stages;           // accumulator buffer, operand slot
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_ACCE0 + s, ((it >> 1) & 1) ^ 1, abort_flag) &&
                                                     tc::mbar_wait(bars + B_FULL0 + sl, (it / stages) & 1, abort_flag));
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t bt = sbase + (uint32_t)(sl * STAGE);
                    if (tc::elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            tc::mma_ss(tmem + (uint32_t)s * acc_cols, tc::desc_kmajor_sw128(bt + (ks >> 2) * (B_TILE / 2), (ks & 3) * 16),
                                       tc::desc_kmajor_sw128(ct + (uint32_t)((ks >> 2) * n_pad * 128), (ks & 3) * 16), idesc, ks != 0);
                        for (int ks = 0; ks < kd_steps; ++ks)      // D = U V^T into the second half of the buffer
                            tc::mma_ss(tmem + (uint32_t)s * acc_cols + 128u, tc::desc_kmajor_sw128(bt + B_TILE, ks * 16),
                                       tc::desc_kmajor_sw128(ct + (uint32_t)c_only, ks * 16), idesc, ks != 0);
                        tc::mma_commit(bars + B_EMPTY0 + sl);
                        tc::mma_commit(bars + B_ACCF0 + s);
                        if (k == kr - 1) tc::mma_commit(bars + B_CE0 + cs);     // last product that reads this C buffer
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    } else {
        const int row = warp * 32 + lane;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        bool ok = true;
        int it = 0;
        for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
            const int kr = min(MAX_ITEMS, my_tiles - r0);
            for (int k = 0; k < kr; ++k) totals[k * TI + row] = 0.f;      // each thread only touches its own column
            const int steps = G * kr;
#pragma unroll 1
            for (int j = 0; j < steps; ++j, ++it) {
                const int k = j % kr;
                const int s = it & 1;
                if (!tc::mbar_wait(bars + B_ACCF0 + s, (it >> 1) & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                float r0s = 0.f, r1s = 0.f, r2s = 0.f, r3s = 0.f;
                const uint32_t tP = tmem + lane_base + (uint32_t)s * acc_cols;
#pragma unroll 1
                for (int c = 0; c < n_pad; c += 16) {                     // n_pad is a multiple of 16
                    uint32_t p[16], d[16];
                    tc::tmem_ld16(tP + (uint32_t)c, p);
                    tc::tmem_ld16(tP + 128u + (uint32_t)c, d);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; e += 4) {
                        r0s = fmaf(fabsf(__uint_as_float(p[e])), __uint_as_float(d[e]), r0s);
                        r1s = fmaf(fabsf(__uint_as_float(p[e + 1])), __uint_as_float(d[e + 1]), r1s);
                        r2s = fmaf(fabsf(__uint_as_float(p[e + 2])), __uint_as_float(d[e + 2]), r2s);
                        r3s = fmaf(fabsf(__uint_as_float(p[e + 3])), __uint_as_float(d[e + 3]), r3s);
                    }
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bars + B_ACCE0 + s);
                totals[k * TI + row] += (r0s + r1s) + (r2s + r3s);
            }
            if (ok) {
                for (int k = 0; k < kr; ++k) {
                    const int i = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI + row;
                    if (i < n_vis) scores[(size_t)b * n_vis + i] = totals[k * TI + row] / ((float)n_text * (float)H);
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 5) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 2 * acc_cols); }
}

}  // namespace

bool str_mamba_dyn_importance_tc_supported(const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C) {
    if (s->dtype != STR_BF16 || s->n != NS || n_text < 1 || n_text > MAX_TEXT || n_vis < 1) return false;
    if (3 * (s->H / s->G) > 64) return false;                   // the high/low pairs of a group's heads fill one 64-column tile
    return (((uintptr_t)B | (uintptr_t)C) & 15) == 0;
}

// U [Bz, n_vis, G, 64], V [Bz, n_pad, G, 64]: the bf16 high/low decay weights (n_pad = n_text rounded up to 16).
int str_mamba_dyn_importance_tc(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C,
                                const void *U, const void *V, float *scores, cudaStream_t st) {
    const int n_pad = (n_text + 15) / 16 * 16;
    const size_t fixed = 2 * (size_t)n_pad * 384 + (size_t)MAX_ITEMS * TI * 4 + B_COUNT * 8 + 32;
    int stages = MAX_STAGES;
    while (stages > 2 && fixed + (size_t)stages * STAGE > (size_t)ctx->max_smem_optin) --stages;
    const size_t smem = fixed + (size_t)stages * STAGE;
    if (smem > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tb, tcm, tu, tv;
    int rc = str_make_tmap_3d_bf16_sw128(ctx, &tb, B, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, TI);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tcm, C, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, (uint32_t)n_pad);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tu, U, (uint64_t)s->G * 64, (uint64_t)n_vis, (uint64_t)s->Bz, TI);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tv, V, (uint64_t)s->G * 64, (uint64_t)n_pad, (uint64_t)s->Bz, (uint32_t)n_pad);
    if (rc != STR_OK) return rc;
    rc = str_ensure_smem(ctx, STR_SMEM_MAMBA_DYN_SCORE, mamba_dyn_score_tc_kernel, smem);
    if (rc != STR_OK) return rc;
    const int tiles = ceil_div(n_vis, TI);
    const int per_seq = ceil_div(ctx->sm_count, s->Bz);
    const int kd_steps = ceil_div(3 * (s->H / s->G), 16);
    dim3 grid(tiles < per_seq ? tiles : per_seq, s->Bz);
    mamba_dyn_score_tc_kernel<<<grid, NUM_THREADS, smem, st>>>(tb, tcm, tu, tv, s->H, s->G, n_vis, n_text, n_pad, stages, kd_steps,
                                                              scores, ctx->status_dev);
    return str_launch_ok(ctx);
}
