// Mamba importance score (Eq. 2, decay excluded) on tcgen05 tensor cores, bf16 inputs, d_state 128:
//   s_i = 1/(M G) sum_g dbar_i^g sum_m | b_i^g . c_m^g |
// Persistent CTAs: each owns the 128-token tiles  blockIdx.x, blockIdx.x + gridDim.x, ...  of one sequence
// and walks  group g (outer) x its tiles (inner), so the text rows C^g of a group are fetched once per CTA
// and group instead of once per tile; the running sums of a CTA's tiles stay in shared memory (rounds of
// up to MAX_ITEMS tiles).  Per (group, tile):
//   P = B_tile C_text^T      [128 tokens x M text rows], both operands K-major in shared memory (TMA,
//                            128-byte swizzle), fp32 accumulator in tensor memory (two buffers)
//   r_i = sum_m |P[i,m]|     one thread per token row reads its accumulator row and sums magnitudes
//   s_i += dbar_i^g r_i      dbar = mean of dt over the heads of the group, fp32, applied after the
//                            absolute value (it is positive), never rounded into the operands
// Text rows are the last M rows of the same B / C buffers the scan reads; the text tile is padded to a
// multiple of 16 rows by the TMA's out-of-range zero fill (the text rows end the sequence), and zero rows
// add nothing to the sum.
// Warps: 0-3 row sums (warp w owns TMEM lanes 32w..32w+31), 4 TMA producer (B ring, two C buffers),
// 5 MMA issuer.  Every mbarrier wait is bounded; a give-up records STR_ERR_TIMEOUT and the CTA tears down.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int TI = 128, NS = 128;
constexpr int B_TILE = 32768;                // 128 tokens x 128 bf16, two 64-column halves
constexpr int MAX_TEXT = 256, MAX_STAGES = 4, MAX_ITEMS = 16;
enum { B_FULL0 = 0, B_EMPTY0 = MAX_STAGES, B_CF0 = 2 * MAX_STAGES, B_CE0 = B_CF0 + 2, B_ACCF0 = B_CE0 + 2, B_ACCE0 = B_ACCF0 + 2,
       B_COUNT = B_ACCE0 + 2 };
constexpr int NUM_THREADS = 192;

__global__ void __launch_bounds__(NUM_THREADS, 1)
mamba_score_tc_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_c, int Tlen,
                      int H, int G, int n_vis, int n_text, int n_pad, int stages, const float *__restrict__ dt,
                      float *__restrict__ scores, int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int c_bytes = n_pad * 256;                         // text tile: n_pad rows x 128 bf16
    uint8_t *c_smem = smem + stages * B_TILE;
    float *totals = (float *)(c_smem + 2 * c_bytes);          // [MAX_ITEMS][128] running sums of this CTA's tiles
    uint64_t *bars = (uint64_t *)(totals + MAX_ITEMS * TI);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int tiles = (n_vis + TI - 1) / TI;
    const int my_tiles = (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;     // tiles of this CTA
    const uint32_t acc_cols = n_pad <= 128 ? 128u : 256u;      // columns of one accumulator buffer

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
        tc::prefetch_tmap(&tmap_b); tc::prefetch_tmap(&tmap_c);
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
                    ++c_issued;
                    for (int k = 0; k < kr; ++k, ++it) {
                        const int s = it % stages;
                        if (!tc::mbar_wait(bars + B_EMPTY0 + s, ((it / stages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        const int i0 = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI;
                        uint64_t *fb = bars + B_FULL0 + s;
                        tc::mbar_arrive_expect_tx(fb, B_TILE);
                        tc::tma_load_3d(smem + s * B_TILE, &tmap_b, fb, g * NS, i0, b);
                        tc::tma_load_3d(smem + s * B_TILE + B_TILE / 2, &tmap_b, fb, g * NS + 64, i0, b);
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
                    const uint32_t bt = sbase + (uint32_t)(sl * B_TILE);
                    if (tc::elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            tc::mma_ss(tmem + (uint32_t)s * acc_cols, tc::desc_kmajor_sw128(bt + (ks >> 2) * (B_TILE / 2), (ks & 3) * 16),
                                       tc::desc_kmajor_sw128(ct + (uint32_t)((ks >> 2) * n_pad * 128), (ks & 3) * 16), idesc, ks != 0);
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
        const int hpg = H / G;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float inv_hpg = 1.0f / (float)hpg;
        const bool vec_dt = hpg <= 16 && (hpg & 3) == 0 && (H & 3) == 0 && (reinterpret_cast<uintptr_t>(dt) & 15) == 0;
        bool ok = true;
        int it = 0;
        for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
            const int kr = min(MAX_ITEMS, my_tiles - r0);
            for (int k = 0; k < kr; ++k) totals[k * TI + row] = 0.f;      // each thread only touches its own column
            // dt of step j+1 is fetched while step j is worked on (up to 16 heads per group as four 16-byte
            // loads; other shapes fall back to loads issued at the start of the step)
            const int steps = G * kr;
            float4 nx[4];
            auto fetch = [&](int j) {
                const int g = j / kr, k = j - g * kr;
                const int i = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI + row;
                const float4 *p4 = reinterpret_cast<const float4 *>(dt + ((size_t)b * Tlen + min(i, Tlen - 1)) * H + g * hpg);
#pragma unroll
                for (int q = 0; q < 4; ++q) nx[q] = (4 * q < hpg) ? __ldg(p4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            };
            if (vec_dt) fetch(0);
#pragma unroll 1
            for (int j = 0; j < steps; ++j, ++it) {
                const int g = j / kr, k = j - g * kr;
                const int s = it & 1;
                float dsum;
                if (vec_dt) {
                    dsum = ((nx[0].x + nx[0].y) + (nx[0].z + nx[0].w)) + ((nx[1].x + nx[1].y) + (nx[1].z + nx[1].w)) +
                           ((nx[2].x + nx[2].y) + (nx[2].z + nx[2].w)) + ((nx[3].x + nx[3].y) + (nx[3].z + nx[3].w));
                    if (j + 1 < steps) fetch(j + 1);
                } else {
                    const int i = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI + row;
                    const float *dtr = dt + ((size_t)b * Tlen + min(i, Tlen - 1)) * H + g * hpg;
                    dsum = 0.f;
                    for (int hh = 0; hh < hpg; ++hh) dsum += __ldg(dtr + hh);
                }
                if (!tc::mbar_wait(bars + B_ACCF0 + s, (it >> 1) & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                float r0s = 0.f, r1s = 0.f, r2s = 0.f, r3s = 0.f;
#pragma unroll 1
                for (int c = 0; c < n_pad; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld32(tmem + lane_base + (uint32_t)s * acc_cols + (uint32_t)c, v);
                    tc::tmem_ld_wait();
                    const int lim = (c + 32 <= n_pad) ? 32 : 16;       // n_pad is a multiple of 16
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        if (e < lim) {
                            r0s += fabsf(__uint_as_float(v[e]));     r1s += fabsf(__uint_as_float(v[e + 1]));
                            r2s += fabsf(__uint_as_float(v[e + 2])); r3s += fabsf(__uint_as_float(v[e + 3]));
                        }
                    }
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bars + B_ACCE0 + s);
                totals[k * TI + row] = fmaf(dsum * inv_hpg, (r0s + r1s) + (r2s + r3s), totals[k * TI + row]);
            }
            if (ok) {
                for (int k = 0; k < kr; ++k) {
                    const int i = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI + row;
                    if (i < n_vis) scores[(size_t)b * n_vis + i] = totals[k * TI + row] / ((float)n_text * (float)G);
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

bool str_mamba_importance_tc_supported(const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C) {
    if (s->dtype != STR_BF16 || s->n != NS || n_text < 1 || n_text > MAX_TEXT || n_vis < 1) return false;
    return (((uintptr_t)B | (uintptr_t)C) & 15) == 0;
}

int str_mamba_importance_tc(str_ctx *ctx, const str_ssm_score_shape *s, int n_vis, int n_text, const void *B, const void *C,
                            const float *dt, float *scores, cudaStream_t st) {
    const int n_pad = (n_text + 15) / 16 * 16;
    const size_t fixed = 2 * (size_t)n_pad * 256 + (size_t)MAX_ITEMS * TI * 4 + B_COUNT * 8 + 32;
    int stages = MAX_STAGES;
    while (stages > 2 && fixed + (size_t)stages * B_TILE > (size_t)ctx->max_smem_optin) --stages;
    const size_t smem = fixed + (size_t)stages * B_TILE;
    if (smem > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tb, tcm;
    int rc = str_make_tmap_3d_bf16_sw128(ctx, &tb, B, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, TI);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tcm, C, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, (uint32_t)n_pad);
    if (rc != STR_OK) return rc;
    rc = str_ensure_smem(ctx, STR_SMEM_MAMBA_SCORE, mamba_score_tc_kernel, smem);
    if (rc != STR_OK) return rc;
    const int tiles = ceil_div(n_vis, TI);
    const int per_seq = ceil_div(ctx->sm_count, s->Bz);
    dim3 grid(tiles < per_seq ? tiles : per_seq, s->Bz);
    mamba_score_tc_kernel<<<grid, NUM_THREADS, smem, st>>>(tb, tcm, s->T, s->H, s->G, n_vis, n_text, n_pad, stages, dt, scores,
                                                          ctx->status_dev);
    return str_launch_ok(ctx);
}
